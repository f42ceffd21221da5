"""CPU oracle for the Pilot-Commit rollout path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy restatement (float64 arithmetic unless a
caller asks for float32) of what the rollout hot path computes: the Qwen2/3-style
decoder forward, seeded Gumbel-max sampling at temperature T, the binary reward
rule of the synthetic workloads, the per-group statistics of Eq. 3, the pilot
estimate and filter of Section 3.3, the eviction rule of Section 3.4 and the
group-relative advantage of Section 3.1.

Nothing in the product package imports this directory.  It is used by the tests,
by the smoke check, and by the benchmark's CPU-baseline leg, and it shares no
code with the CUDA path: only the seeded input generators
(`paper_2605_26606_b200.workloads`) serve both sides.

Pins (see tests/test_oracle_*.py): every function here is checked against
something other than itself -- closed forms, invariants the paper states, values
the paper prints, brute force, or an independent library routine.  The one
exception is stated in `oracle/philox.py`.
"""
