"""CPU oracle for the ShotKV hot path (test infrastructure, fp64, slow on purpose).

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product path never does and fails loudly without its CUDA library.
"""
