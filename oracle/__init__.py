"""CPU ORACLE -- test infrastructure, not product code.

A plain, slow, independent CPU statement of what the verification path computes
(decoder forward with and without KV cache, autoregressive and speculative loops, the
accept/reject/resample rule).  Nothing here is shared with, imported by, or imports the CUDA
package.  Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
"""
