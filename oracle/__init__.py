"""Float64 CPU oracle for the Continuous Task Batching (CTB) hot path.

TEST INFRASTRUCTURE ONLY.  This package is the slow, plain definition of what
the CUDA library computes: a paged KV cache with a deterministic page
allocator, the append of resumed tasks' observation tokens, and grouped-query
softmax attention of a mixed decode / resume batch over the preserved cache
(the state CTB keeps resident across environment pauses, paper Section 4 and
Algorithm 1).  Only the tests, the smoke check and the CPU-baseline leg of the
benchmark may import it.  It shares no code with the CUDA path and never
imports it.

Modules
  paged_kv   page allocator + logical cache (bit-exact integer / byte work)
  attention  float64 attention, brute-force variant, log-sum-exp merge
  cbuild     builds and loads csrc/attend_f64.c (same maths in plain C with
             OpenMP, for workloads too large for numpy)

Parity pins: every function here is pinned by tests/test_oracle_*.py against
brute force, closed forms and invariants; nothing is "parity unpinned".
"""
