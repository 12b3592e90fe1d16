"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot replay a whole rollout of these shapes, so it scores sampled sequences teacher-
forced along the GPU's own tokens (layer-streamed), and the rest is covered by properties that
hold at any size: page table bit-exact, version tags, log-probabilities non-positive, and the
teacher-forced entry point reproducing the free-running log-probabilities at every step.
"""
import os

import numpy as np
import pytest
import torch

from oracle import pages
from paper_2602_02192_b200 import synth
from helpers import LOGPROB_TOL, MARGIN_EXEMPT, StreamedWeights, dims_of, score_sequences

pytestmark = pytest.mark.gpu

# (workload, sequences scored by the oracle, decode steps scored).  The 32B shape (65 GB of weights
# generated into page-locked host memory, a 64-layer oracle pass over 1032 positions) takes about four
# minutes on its own; ECHO_TEST_SKIP_32B=1 leaves it out, and it is skipped on a host with less than
# 100 GB of free memory.
CASES = [("0.6B", [0, 257], 1024), ("4B", [5, 100], 32), ("8B", [3, 200], 32)]
if os.environ.get("ECHO_TEST_SKIP_32B") != "1":
    CASES += [("32B", [1], 8)]


@pytest.mark.parametrize("name,seqs,steps", CASES)
def test_full_size_rollout(name, seqs, steps):
    from paper_2602_02192_b200 import binding as B
    wl = synth.WORKLOADS[name]
    shape, P, G, Lp, T = wl.shape, wl.n_prompts, wl.G, wl.prompt_len, wl.new_tokens
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    free, total = torch.cuda.mem_get_info()
    cfg = B.make_config(shape, P, G, Lp, T, 1, half_layers=wl.half_layers)     # as bench.py runs it
    on_host = 2 * shape.n_params() > 40e9              # snapshot kept in pinned host memory
    if on_host:
        import psutil
        if psutil.virtual_memory().available < 100e9:
            pytest.skip("needs 100 GB of free host memory for the snapshot and the oracle's layers")
    need = B.echo_arena_bytes(cfg) + (0 if on_host else 2 * shape.n_params()) + (2 << 30)
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of device memory")
    eng = B.Engine(cfg)
    w = (synth.make_weights_pinned(shape, wl.weight_seed) if on_host
         else synth.make_weights(shape, wl.weight_seed, device="cuda"))
    eng.echo_load_policy(w, 3)
    prompts = synth.make_prompts(P, Lp, shape.vocab, wl.prompt_seed)
    dp = torch.from_numpy(prompts).cuda()
    lens = [Lp] * P
    tok, lp, ver = eng.echo_rollout(dp, lens, G, T, wl.temperature, wl.sample_seed)
    eng.echo_sync()
    assert np.all(ver == 3)
    plan = pages.build(lens, G, T, 16)
    got = eng.echo_debug_page_table()
    assert np.array_equal(got[:, : plan.width], plan.table) and eng.echo_get_stats()["n_pages"] == plan.n_pages
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    assert tok_h.min() >= 0 and tok_h.max() < shape.vocab and np.all(lp_h <= 0) and np.all(np.isfinite(lp_h))
    # random-init logits are nearly flat: the mean log-probability sits near -log(V)
    assert abs(lp_h.mean() + np.log(shape.vocab)) < 1.5
    # Teacher-forced replay of the GPU's own tokens reproduces its log-probabilities at every step.
    # With ECHO_DETERMINISTIC=1 (fixed-order reductions) bit for bit.  By default the split
    # projections add their k-slices in whatever order the CTAs finish; a last-bit difference that
    # flips the 16-bit rounding of an activation or a cached key decorrelates the later roundings, so
    # two runs differ from each other about as much as either differs from exact arithmetic.
    tok_f, lp_f, _ = eng.echo_rollout(dp, lens, G, T, wl.temperature, wl.sample_seed, forced=tok)
    eng.echo_sync()
    dlp = np.abs(lp_f.cpu().numpy() - lp_h)
    print(f"{name}: free run vs teacher-forced replay: mean {dlp.mean():.2e} q99.9 {np.quantile(dlp, 0.999):.2e} "
          f"max {dlp.max():.2e} same tokens {(tok_f.cpu().numpy() == tok_h).mean():.4f}")
    if os.environ.get("ECHO_DETERMINISTIC") == "1":
        assert dlp.max() == 0.0 and np.array_equal(tok_f.cpu().numpy(), tok_h)
    else:
        # measured on B200: mean 1.7e-3 / 7.0e-3 / 8.0e-3 and 99.9 % below 7.0e-3 / 2.9e-2 / 3.3e-2 at the
        # 0.6B / 4B / 8B shapes, 99.4 % or more of the tokens equal (32B: 8.8e-3, 3.7e-2, 99.4 %)
        assert dlp.mean() < 1.5e-2 and np.quantile(dlp, 0.999) < 6.5e-2, (dlp.mean(), dlp.max())
        assert (tok_f.cpu().numpy() == tok_h).mean() > 0.985
    # sampled sequences against the oracle: the acceptance rule, token by token
    sw = StreamedWeights(w)
    delta, same, second, margin = score_sequences(dims_of(shape), sw, prompts, lens, G, wl.temperature,
                                                  wl.sample_seed, tok_h, lp_h, seqs, steps=steps,
                                                  layer_provider=sw.layer)
    print(f"{name}: half_layers={wl.half_layers} n={delta.size} mean|dlp|={delta.mean():.4f} "
          f"median={np.median(delta):.4f} max={delta.max():.4f} within_tol={(delta <= LOGPROB_TOL).mean():.3f} "
          f"token_match={same.mean():.3f} exempt={int((~same).sum())}")
    assert delta.size == len(seqs) * steps
    assert delta.max() <= LOGPROB_TOL
    bad = ~same
    assert np.all(second[bad]) and np.all(margin[bad] < MARGIN_EXEMPT) and bad.sum() <= max(2, 0.05 * delta.size)
    eng.close()
