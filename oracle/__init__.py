"""LoCo oracle: test infrastructure, not the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this
package.  It does not import, link or read anything of the CUDA library.
"""
