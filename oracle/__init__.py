"""CPU oracle: plain, slow, obviously-correct reference implementations.

TEST INFRASTRUCTURE ONLY.  Nothing in the library or its Python binding may import this
package; it exists so that tests, the smoke check and the benchmark's CPU-baseline leg can
compare the GPU path with the definitions.
"""
