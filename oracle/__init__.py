"""CPU oracle for the S2D2 draft-then-verify decode step.

TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 restatement of what the decode
step computes, written from the paper's algorithms (block-wise decoding loop,
the S2D2 block sampler, the verifier and drafting masks, the speculative
acceptance rule).  It shares no code with the CUDA path and must never be
imported by the product package: only the tests, the smoke check and the
bench's CPU-baseline leg call it.

Pins (what each part is checked against, see tests/test_oracle_*.py):
  philox.py   published known-answer vectors of Philox4x32-10.
  model.py    a separately written composition of torch fp64 library ops for a
              plain causal pass; RoPE shift invariance; cached == recomputed;
              MoE top-k == dense evaluation with zeroed gates; K/V of bf16 models held
              as bfloat16 (the cache's storage format): nearest bfloat16 of the fp64 value,
              ties to even, == torch's bfloat16 conversion on fp32 inputs.
  accept.py   scipy logsumexp; closed forms of speculative sampling (exact
              enumeration on tiny vocabularies); brute-force inverse CDF.
  s2d2.py     draft rows == Eq. (draft_mask) block by block for every first masked position and
              every cached prefix, and draft logits on a cache == one literal pass over
              prompt ++ block under the composed mask (three wrong masks fail both);
              verifier rows of the 2L pass == L literal single-row passes;
              block size 1 == greedy autoregressive decoding; committed K/V ==
              K/V of a final causal pass over the finished block.
  routing.py  hand-computed values of the expected accepted prefix length.

Parity unpinned (no statement in the paper fixes them): the points at which
the CUDA path rounds to bfloat16, the "mean draft confidence < 0.9" routing
rule of the 4B-class workload, and absolute token trajectories.
"""
