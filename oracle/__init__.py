"""CPU oracle for the d2Cache decode step.  TEST INFRASTRUCTURE, NOT PRODUCT.

A plain, slow numpy implementation (fp64 arithmetic, fp32 where the method's
state is fp32) of what one d2Cache decoding step computes, written from the
paper's equations (Sections 3.1 and 4, Eq. 1-9).  Only the tests, the smoke
check and the benchmark's CPU-baseline leg may import it.  It shares no code
with the CUDA path and imports nothing from the product package.

Pin status (see tests/test_oracle_*.py):
  selection.density / density_q30     closed forms + brute force
  selection.stage1 / stage2           rank-counting and exhaustive-subset brute force
  rollout.literal / rollout.chain     each other, N=1 and uniform-attention closed forms, sum = L
  model.* (select-all)                an independently written torch fp64 textbook forward
  model.lm_head_conf                  softmax identities, zero-weight closed form
  step.oracle_step                    select-all == no-cache forward; select-none == identity;
                                      single-layer exactness; a strict subset of rows on two and
                                      three layers with a stale cache == an independently written
                                      torch fp64 subset step (index assignment into the cache, library
                                      attention over all keys); rollout_layers = n == Eq. 6-9 over the
                                      first n layers of the same step (and differs from the last n)
"""
