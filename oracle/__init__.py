"""CPU oracle -- test infrastructure only.

Plain, slow, obviously-correct implementations of what the token-mask path computes.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the product
package never does, and nothing here imports the product's binding.
"""
