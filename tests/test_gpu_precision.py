"""Where the 16-bit path's error enters, measured inside the engine at the 8B width.

Two checks that stand beside the full-size parity test:

* one layer at a time, NOT compounding: the engine records the residual stream as it enters and
  leaves a layer (echo_debug_capture); the oracle's layer is applied to the engine's own input and
  the two outputs are compared.  A wrong kernel, index or weight shows here at its layer, whatever
  the layers before it did.
* depth sweep: the same width with 2, 4, 9, 18, 36 layers, log-probabilities against the oracle.
  A defect in one kernel would show as a floor at two layers or as a jump at some depth; rounding
  error shows as a smooth curve.  With bf16 operands everywhere the curve crosses the 5e-2 bound
  near full depth; with the first layers' operands in IEEE half (echo_config.half_layers) it stays
  below it at every depth, which is the configuration the benchmark runs.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import decoder
from paper_2602_02192_b200 import synth
from helpers import LOGPROB_TOL, MARGIN_EXEMPT, StreamedWeights, dims_of

pytestmark = pytest.mark.gpu

P, G, LP = 32, 8, 64            # 256 rows per decode step, as in the benchmark


@pytest.fixture(scope="module")
def B():
    from paper_2602_02192_b200 import binding
    return binding


@pytest.fixture(scope="module")
def w8b():
    wl = synth.WORKLOADS["8B"]
    import gc
    gc.collect()
    torch.cuda.empty_cache()                 # blocks cached from the tests before count as used otherwise
    free, _ = torch.cuda.mem_get_info()
    if free < 60e9:
        pytest.skip("needs 60 GB of device memory")
    w = synth.make_weights(wl.shape, wl.weight_seed, device="cuda")
    return wl, w, StreamedWeights(w)


def _truncated(w, n_layers):
    return {k: (v[:n_layers] if isinstance(v, list) else v) for k, v in w.items()}


@pytest.mark.parametrize("half_layers", [0, 4])
def test_single_layers_against_the_oracle_on_the_engines_own_input(B, w8b, half_layers):
    wl, w, sw = w8b
    shape = wl.shape
    T = 5
    d = shape.d_model
    eng = B.Engine(B.make_config(shape, P, G, LP, T, 1, half_layers=half_layers))
    eng.echo_load_policy(w, 1)
    prompts = synth.make_prompts(P, LP, shape.vocab, wl.prompt_seed)
    dp = torch.from_numpy(prompts).cuda()
    bufs = [torch.zeros((P * LP, d), device="cuda") for _ in range(2)] + \
           [torch.zeros((T - 1, P * G, d), device="cuda") for _ in range(2)]
    dims = dims_of(shape)
    report = {}
    for layer in (0, 1, 17, 35):
        eng.echo_debug_capture(layer, *bufs)
        eng.echo_rollout(dp, [LP] * P, G, T, 1.0, wl.sample_seed)
        eng.echo_sync()
        pre_in, pre_out, dec_in, dec_out = (b.cpu().numpy().astype(np.float64) for b in bufs)
        lw = sw.layer(layer)
        for s in (1, 130):                                   # sequence (p, g): prompt rows, then its decode rows
            p = s // G
            x_in = np.concatenate([pre_in[p * LP:(p + 1) * LP], dec_in[:, s]])
            got = np.concatenate([pre_out[p * LP:(p + 1) * LP], dec_out[:, s]])
            want = decoder.layer_sequence(dims, lw, x_in)
            step = want - x_in                               # what the layer adds to the residual stream
            scale = np.sqrt(np.mean(step ** 2))
            err = got - want
            for name, rows in (("prefill", slice(0, LP)), ("decode", slice(LP, LP + T - 1))):
                rel_rms = np.sqrt(np.mean(err[rows] ** 2)) / scale
                rel_max = np.max(np.abs(err[rows])) / scale
                report[(layer, s, name)] = (rel_rms, rel_max)
                # Bounds = 1.4 x what B200 measures (the table this test prints): a layer with bf16
                # operands is off by 3.0e-3 to 3.5e-3 of the rms of what it adds (worst element 1.8e-2),
                # one with half operands by 4e-4 to 1e-3.  Layer 0 is off by 8e-3 with bf16 operands:
                # its MLP normalises a residual stream that consists of the attention output alone,
                # which multiplies the attention block's rounding error inside that layer.
                if layer < half_layers:
                    lim_rms, lim_max = 1.5e-3, 6.5e-3
                elif layer == 0:
                    lim_rms, lim_max = 1.1e-2, 5.5e-2
                else:
                    lim_rms, lim_max = 4.8e-3, 2.5e-2
                assert rel_rms < lim_rms, (layer, s, name, rel_rms)
                assert rel_max < lim_max, (layer, s, name, rel_max)
    eng.echo_debug_capture(-1)
    eng.close()
    for k, v in sorted(report.items()):
        print(f"half_layers={half_layers} layer {k[0]:2d} seq {k[1]:3d} {k[2]:7s} rms err / rms step = {v[0]:.3e}  max = {v[1]:.3e}")


def test_error_against_depth(B, w8b):
    wl, w, sw = w8b
    T = 12
    seqs = [3, 200]
    prompts = synth.make_prompts(P, LP, wl.shape.vocab, wl.prompt_seed)
    dp = torch.from_numpy(prompts).cuda()
    lens = [LP] * P
    curve = {}
    for L in (2, 4, 9, 18, 36):
        shape = dataclasses.replace(wl.shape, n_layers=L)
        wL = _truncated(w, L)
        lp = {}
        tok = would = None
        for hl in (0, min(wl.half_layers, L)):
            eng = B.Engine(B.make_config(shape, P, G, LP, T, 1, half_layers=hl))
            eng.echo_load_policy(wL, 1)
            t, l, _ = eng.echo_rollout(dp, lens, G, T, 1.0, wl.sample_seed, forced=tok)
            eng.echo_sync()
            if tok is None:
                tok = t
            else:
                would = t.cpu().numpy()
            lp[hl] = l.cpu().numpy()
            eng.close()
        tok_h = tok.cpu().numpy()
        hl = min(wl.half_layers, L)
        d_bf16, d_half = [], []
        for s in seqs:
            p, g = divmod(s, G)
            sc = decoder.score_forced(dims_of(shape), sw, prompts[p], tok_h[p, g], 1.0, wl.sample_seed, s,
                                      layer_provider=sw.layer)
            d_bf16.append(np.abs(lp[0][p, g] - sc.logprob_given))
            d_half.append(np.abs(lp[hl][p, g] - sc.logprob_given))
            # the configuration the benchmark runs meets the acceptance rule at every depth
            assert np.max(d_half[-1]) <= LOGPROB_TOL, (L, s, np.max(d_half[-1]))
            for j in range(T):
                y = int(would[p, g, j])
                assert y == sc.own_token[j] or (sc.margin[j] < MARGIN_EXEMPT and y == sc.runner_up[j]), (L, s, j)
        curve[L] = (float(np.mean(d_bf16)), float(np.max(d_bf16)), float(np.mean(d_half)), float(np.max(d_half)))
        print(f"layers {L:2d}: bf16 everywhere mean {curve[L][0]:.3e} max {curve[L][1]:.3e} | "
              f"half_layers={hl} mean {curve[L][2]:.3e} max {curve[L][3]:.3e}")
    depths = sorted(curve)
    for a, b in zip(depths, depths[1:]):
        # from one depth to the next (x 2, once x 2.25) the mean error grows at most a little faster than
        # the depth and never falls by much: a curve, not a step.  Measured ratios: 1.1-2.7 with bf16
        # everywhere (the largest from 4 to 9 layers, 2.55-2.64 in different runs: the order of the split
        # projections' sums varies), 1.1-1.8 with half layers.
        for col in (0, 2):
            r = curve[b][col] / curve[a][col]
            assert 0.6 < r < 1.4 * b / a, (a, b, col, r)
    assert curve[36][2] < 0.5 * curve[36][0]                  # what the half layers buy at full depth
