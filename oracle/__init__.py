"""CPU oracle for the all-boundary draft step (TEST INFRASTRUCTURE, not a product path).

Plain numpy, float64 arithmetic unless a function says otherwise, one obvious loop nest per
definition, written from the paper's description of the method.  Nothing here is imported by the
CUDA package, and nothing here imports it.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may call into this package.

Modules
-------
attention : every acceptance boundary as an independent plain softmax attention (paper Sec. 3.2,
            Fig. 4: shared causal spine, isolated bidirectional branches, all rows read the cache).
verify    : accepted length, bonus token and branch selection (paper Sec. 2.1, Alg. 1 lines 2-3,
            App. C for the rejection rule).
layer     : one drafter backbone block around the attention (paper Sec. 3.1 only lists a block's
            parts -- attention, MLP, norms; the block structure is this build's reading
            -- PARITY UNPINNED by the paper for the structure itself, pinned only piecewise).
cache     : the feature-cache update of Alg. 1 (verified rows appended, rejected suffix dropped) as keys/values of
            every drafter layer, row by row.
"""
from . import attention, verify, layer, cache  # noqa: F401
