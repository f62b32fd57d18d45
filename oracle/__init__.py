"""CPU checker for the TABED speculative-decoding round.

TEST INFRASTRUCTURE ONLY: slow, plain and written from the paper.  It shares no
code with the CUDA library and must never be imported by the product path; only
tests, the smoke check and the benchmark's CPU-baseline leg use it.

definitions.py  fp64 textbook definitions (softmax, ensemble, KL, TVD, acceptance, policies, Eq. 1)
exact32.py      the integer-deciding arithmetic in the kernel's precision (fp32 + exact integers)
drafter.py      fp64 forward pass of the shared LLaMA-style drafter, one row at a time
tabed.py        Algorithm 1 + verification + weight update as a per-request state machine

Pin status: every function is pinned by tests that do not retype its formula
(closed forms, invariants, brute-force enumeration, library routines); the
numerical VALUES of the adapted weights are "parity unpinned" by the paper (it
prints no worked example) and rest on the readings listed in the design notes.
"""
