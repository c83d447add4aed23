"""CPU oracle of the 2:4 masked convolution path (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package; the CUDA library and its Python binding never do, and this package never
imports them.
"""
