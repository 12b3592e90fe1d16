"""CPU oracle for GRPO rollout generation.  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Plain, slow, obviously-correct numpy (fp64) restatement of what the rollout hot
path computes: a decoder-only transformer sampled G times per prompt with
Philox-keyed Gumbel-max, per-token log-probabilities of the sampling
distribution, a version tag per trajectory, and GRPO's group-normalised rewards.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA path and imports nothing from it.

Pins (what each function is checked against, other than itself) are listed in
the docstring of each module; a function without one says "parity unpinned".
"""
