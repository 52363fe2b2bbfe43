"""CPU oracle for one SPACE auto-correct decoding step (arXiv 2402.11809).

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain, fp64 statement of
what the step computes, written from the paper.  It shares no code with the
CUDA library and must never be imported by it.  Only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may call it.

Modules
-------
layout     block rows, visibility rule (Eq. 5 and the Sec. 3.2 / App. A.3 text),
           position ids (Sec. 3.2)
brute      full |I| x |I| masked attention straight from Eq. 4 / Eq. 5 (tiny sizes)
attention  block-over-cache attention in fp64
philox     Philox4x32-10 counter-based generator (Salmon et al., SC'11)
verify     Algorithm 1 verification: greedy and rejection sampling
commit     compaction of accepted rows into the verified cache
lmhead     output projection (hidden states x output embedding) followed by greedy
           verification: the end of the model call of Algorithm 1 and the loop after it
bf16       exact bf16 <-> float conversion helpers

Parity pins: every function here is pinned by a CPU test (tests/test_oracle_*.py);
no function is "parity unpinned".
"""
