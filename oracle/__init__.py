"""CPU oracle for the VC-Attention hot path -- TEST INFRASTRUCTURE, not product code.

A plain, slow NumPy restatement of what the path computes, written from the paper:

* ``codecs``     number formats (E4M3, E2M1, bf16) and the ExpCast-FP8 map (Eq. 7)
* ``prep``       the preprocessing chain (Sec. 3.4 "Fused preprocessing", App. B)
* ``attention``  exact fp64 attention and the emulated low-bit recurrence
                 (Eq. 1, Eq. 6, Eq. 7)
* ``grouping``   the value-guided permutation (Sec. 3.2): k-means labels, stable argsort
* ``analysis``   analogues of the paper's value-side analysis (token-order table, Eq. 2, Eq. 5)

Only the tests, ``__graft_entry__.smoke()`` and the ``cpu_baseline`` / ``--impl reference``
legs of ``bench.py`` may import this package.  It shares no code with the CUDA path and
never imports it.

Pins (tests/test_oracle_*.py): the codecs are pinned exhaustively and against an
independent library cast; Hadamard, K smoothing, permutation, block demeaning and mean
restoration are pinned by the identities the paper states for them; ExpCast-FP8 by the
paper's worked example and printed constants; the recurrence by brute-force attention
with quantization switched off; every block quantizer (8-bit Q/K blocks, NVFP4 groups under an
outer scale, the NVFP4 probability format, the quantized branches of the V pass) by Python
loops and a brute-force nearest-value search on inputs with planted maxima and ties
(tests/test_oracle_quantizers.py).  The *end-to-end quantized* output has no printed value
in the paper: "parity unpinned" for the granularity of the Q/K scales, the NVFP4
second-level scales and the RoPE channel split, which are readings fixed by this build.
Grouping is pinned by brute-force nearest-centroid search, cluster recovery on separated
blobs, the monotone k-means objective and the definition of a stable sort; k, the
initialisation and the iteration count are readings too ("parity unpinned").
"""
