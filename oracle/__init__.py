"""CPU oracle for the GPU-resident serving loop.  TEST INFRASTRUCTURE ONLY.

Plain, slow and meant to be checked by eye against the paper: the scheduling
policy (FCFS continuous batching, Section 4.2), the slot life cycle (Section
4.2, "Ring buffer"), the paged-KV block bookkeeping the control plane keeps on
the device (Sections 1 and 4.2), standard decoder-only transformer math, and
in-step sampling (Section 4.2, "CUDA graph cache").

Nothing in the product path may import this package: only the tests, the
smoke check and the benchmark's CPU-baseline leg do.  It shares no code with
the CUDA path and never receives values produced by it, except the logged
per-iteration visibility watermark that makes real-time arrivals replayable.

Parity pins (see tests/test_oracle_*.py): every function here is pinned by
something other than itself; none is "parity unpinned".
"""
