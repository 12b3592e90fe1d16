"""End-to-end GPU rollouts against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import decoder, pages
from paper_2602_02192_b200 import synth
from helpers import LOGPROB_TOL, assert_same_rollout, check_sequences, dims_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_02192_b200 import binding
    return binding


@pytest.fixture(scope="module")
def tiny(B):
    wl = synth.WORKLOADS["tiny"]
    w_t = synth.make_weights(wl.shape, wl.weight_seed)
    w_o = decoder.Weights(synth.weights_to_bits(w_t))
    w_d = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w_t.items()}
    return wl, w_o, w_d


def _engine(B, shape, P, G, Lp, T, nbuf=2):
    return B.Engine(B.make_config(shape, P, G, Lp, T, nbuf))


def test_tiny_config_full_parity(B, tiny):
    wl, w_o, w_d = tiny
    eng = _engine(B, wl.shape, wl.n_prompts, wl.G, wl.prompt_len, wl.new_tokens)
    eng.echo_load_policy(w_d, 5)
    prompts = synth.make_prompts(wl.n_prompts, wl.prompt_len, wl.shape.vocab, wl.prompt_seed)
    lens = [wl.prompt_len] * wl.n_prompts
    tok, lp, ver = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, wl.G, wl.new_tokens,
                                    wl.temperature, wl.sample_seed)
    eng.echo_sync()
    tok, lp = tok.cpu().numpy(), lp.cpu().numpy()
    assert np.all(ver == 5)
    # page table: bit-exact against the oracle's plan
    plan = pages.build(lens, wl.G, wl.new_tokens, 16)
    got = eng.echo_debug_page_table()
    assert got.shape[0] == wl.n_prompts * wl.G
    assert np.array_equal(got[:, : plan.width], plan.table)
    assert np.all(got[:, plan.width:] == -1)
    assert eng.echo_get_stats()["n_pages"] == plan.n_pages
    n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, wl.G, wl.temperature, wl.sample_seed,
                                   tok, lp, range(wl.n_prompts * wl.G))
    assert n == wl.n_prompts * wl.G * wl.new_tokens
    assert ex <= 0.05 * n
    assert np.all(lp <= 0)
    # samples of one group differ, and the run is reproducible
    assert len({tuple(tok[0, g]) for g in range(wl.G)}) == wl.G
    tok2, lp2, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, wl.G, wl.new_tokens,
                                    wl.temperature, wl.sample_seed)
    eng.echo_sync()
    assert_same_rollout(tok2.cpu().numpy(), lp2.cpu().numpy(), tok, lp)
    st = eng.echo_get_stats()
    assert st["tokens_generated"] == tok.size and st["kernels_launched"] > 100
    eng.close()


def test_end_of_sequence_rule(B, tiny):
    """eos_id set: a sequence that emits the end token holds eos / log-probability 0 from then on,
    everything else is unchanged; checked against the oracle's rule, free-running and teacher-forced."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 3, 3, 20, 12
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 77)
    lens = [Lp, Lp - 3, Lp]
    dp = torch.from_numpy(prompts).cuda()
    eng = _engine(B, wl.shape, P, G, Lp, T)
    eng.echo_load_policy(w_d, 1)
    tok0, lp0, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 123)
    eng.echo_sync()
    tok0 = tok0.cpu().numpy()
    eng.close()
    eos = int(tok0[1, 1, 4])
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, eos_id=eos))
    eng.echo_load_policy(w_d, 1)
    tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 123)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 123, tok_h, lp_h, range(P * G),
                                   eos_id=eos)
    assert n == P * G * T and ex <= 2
    e = int(np.flatnonzero(tok_h[1, 1] == eos)[0])
    assert e <= 4 and np.all(tok_h[1, 1, e:] == eos) and np.all(lp_h[1, 1, e + 1:] == 0.0) and lp_h[1, 1, e] < 0
    # teacher-forced along that trajectory: finished positions score 0 and "would sample" eos
    tok_f, lp_f, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 123, forced=tok)
    eng.echo_sync()
    tok_f, lp_f = tok_f.cpu().numpy(), lp_f.cpu().numpy()
    fin = np.zeros_like(tok_h, dtype=bool)
    fin[..., 1:] = np.logical_or.accumulate(tok_h[..., :-1] == eos, axis=-1)
    assert np.all(lp_f[fin] == 0.0) and np.all(tok_f[fin] == eos)
    assert np.max(np.abs(lp_f - lp_h)[~fin]) < LOGPROB_TOL
    eng.close()


def test_top_p_rollout(B, tiny):
    """Nucleus sampling inside the engine (config top_p): every token and renormalised log-probability
    against the oracle, teacher-forced along the GPU's tokens; a smaller top_p gives log-probabilities
    that are never lower than the untruncated ones for the same tokens."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 3, 4, 24, 10
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 31)
    lens = [Lp, Lp - 5, Lp]
    dp = torch.from_numpy(prompts).cuda()
    top_p = 0.9
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, top_p=top_p))
    eng.echo_load_policy(w_d, 1)
    tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 2024)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 2024, tok_h, lp_h, range(P * G),
                                   top_p=top_p)
    assert n == P * G * T and ex <= 0.05 * n and np.all(lp_h <= 0)
    eng.close()
    # the same tokens scored without truncation: log p - log(nucleus mass) >= log p
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T))
    eng.echo_load_policy(w_d, 1)
    _, lp_full, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 2024, forced=tok)
    eng.echo_sync()
    d = lp_h - lp_full.cpu().numpy()
    assert np.all(d > -1e-3) and np.all(d < -np.log(top_p) + 5e-2) and d.mean() > 0.02
    eng.close()


def test_forced_rollout_scores_oracle_trajectory(B, tiny):
    wl, w_o, w_d = tiny
    P, G, Lp, T = 2, 3, 20, 12                    # Lp not a multiple of the page size
    eng = _engine(B, wl.shape, P, G, 24, T)
    eng.echo_load_policy(w_d, 0)
    prompts, lens = synth.make_ragged_prompts([20, 13], wl.shape.vocab, 77, pad_to=24)
    ref = decoder.rollout_cached(dims_of(wl.shape), w_o, prompts, lens, G, T, 1.0, 31)
    forced = torch.from_numpy(ref.tokens).cuda()
    tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 31, forced=forced)
    eng.echo_sync()
    tok, lp = tok.cpu().numpy(), lp.cpu().numpy()
    assert np.max(np.abs(lp - ref.logprobs)) <= 5e-2
    diff = tok != ref.tokens
    assert np.all(ref.margins[diff] < 1e-2) and np.all(tok[diff] == ref.runner_up[diff])
    # page plan with ragged, non-page-aligned prompts
    plan = pages.build(lens, G, T, 16)
    got = eng.echo_debug_page_table()
    assert np.array_equal(got[:, : plan.width], plan.table)
    # free-running rollout on the same ragged prompts follows the acceptance rule too
    tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 31)
    eng.echo_sync()
    check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 31, tok.cpu().numpy(), lp.cpu().numpy(),
                    range(P * G))
    eng.close()


def test_edge_shapes(B, tiny):
    wl, w_o, w_d = tiny
    eng = _engine(B, wl.shape, 3, 5, 40, 9)
    eng.echo_load_policy(w_d, 1)
    for P, G, T, lens in [(1, 1, 1, [1]), (1, 2, 2, [16]), (3, 5, 9, [40, 17, 1]), (2, 1, 3, [33, 32])]:
        prompts, lens_a = synth.make_ragged_prompts(lens, wl.shape.vocab, 5 + P, pad_to=40)
        tok, lp, ver = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens_a, G, T, 0.8, 1234)
        eng.echo_sync()
        assert tok.shape == (P, G, T) and np.all(ver == 1)
        check_sequences(dims_of(wl.shape), w_o, prompts, lens_a, G, 0.8, 1234, tok.cpu().numpy(),
                        lp.cpu().numpy(), range(P * G))
    # argument errors
    prompts = torch.zeros((1, 40), dtype=torch.int32, device="cuda")
    for kwargs in [dict(G=6), dict(T=10), dict(temp=0.0), dict(lens=[41]), dict(lens=[0])]:
        with pytest.raises(B.EchoError) as ei:
            eng.echo_rollout(prompts, kwargs.get("lens", [5]), kwargs.get("G", 2), kwargs.get("T", 3),
                             kwargs.get("temp", 1.0), 0)
        assert ei.value.code == -1
    # an out-of-range token id is reported, not trapped on
    bad = torch.full((1, 40), wl.shape.vocab + 3, dtype=torch.int32, device="cuda")
    eng.echo_rollout(bad, [4], 1, 2, 1.0, 0)
    with pytest.raises(B.EchoError) as ei:
        eng.echo_sync()
    assert ei.value.code == -7
    eng.echo_sync()                                  # status is cleared; the context stays usable
    eng.close()


def test_versions_and_double_buffer(B, tiny):
    wl, w_o, w_d = tiny
    w1_t = synth.make_weights(wl.shape, 1)
    w1_o = decoder.Weights(synth.weights_to_bits(w1_t))
    w1_d = {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w1_t.items()}
    P, G, Lp, T = 2, 2, 16, 6
    eng = _engine(B, wl.shape, P, G, Lp, T)
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 3)
    dp = torch.from_numpy(prompts).cuda()
    with pytest.raises(B.EchoError) as ei:
        eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 0)
    assert ei.value.code == -3                        # no policy yet
    eng.echo_load_policy(w_d, 10)
    with pytest.raises(B.EchoError) as ei:
        eng.echo_load_policy(w1_d, 11)
    assert ei.value.code == -5                        # first install not yet picked up
    t0, l0, v0 = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 7)
    assert np.all(v0 == 10)
    with pytest.raises(B.EchoError) as ei:
        eng.echo_load_policy(w1_d, 10)
    assert ei.value.code == -4                        # versions strictly increase
    eng.echo_load_policy(w1_d, 11)
    eng.echo_wait_policy()
    t1, l1, v1 = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 7)
    assert np.all(v1 == 11)
    eng.echo_sync()
    d = dims_of(wl.shape)
    check_sequences(d, w_o, prompts, [Lp] * P, G, 1.0, 7, t0.cpu().numpy(), l0.cpu().numpy(), range(P * G))
    check_sequences(d, w1_o, prompts, [Lp] * P, G, 1.0, 7, t1.cpu().numpy(), l1.cpu().numpy(), range(P * G))
    assert not np.array_equal(t0.cpu().numpy(), t1.cpu().numpy())
    # a third snapshot goes back into the first buffer while version 11 serves
    eng.echo_load_policy(w_d, 12)
    eng.echo_wait_policy()
    t2, l2, v2 = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 7)
    eng.echo_sync()
    assert np.all(v2 == 12)
    assert_same_rollout(t2.cpu().numpy(), l2.cpu().numpy(), t0.cpu().numpy(), l0.cpu().numpy())
    eng.close()
    # single buffer: the next rollout waits for the install and serves the new version
    eng = _engine(B, wl.shape, P, G, Lp, T, nbuf=1)
    eng.echo_load_policy(w_d, 0)
    ta, la, va = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 7)
    eng.echo_load_policy(w1_d, 1)
    tb, lb, vb = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 7)
    eng.echo_sync()
    assert np.all(va == 0) and np.all(vb == 1)
    assert_same_rollout(ta.cpu().numpy(), la.cpu().numpy(), t0.cpu().numpy(), l0.cpu().numpy())
    assert_same_rollout(tb.cpu().numpy(), lb.cpu().numpy(), t1.cpu().numpy(), l1.cpu().numpy())
    eng.close()


def test_host_buffer_entry_point(B, tiny):
    wl, w_o, w_d = tiny
    P, G, Lp, T = 2, 2, 16, 5
    eng = _engine(B, wl.shape, P, G, Lp, T)
    eng.echo_load_policy(w_d, 0)
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 8)
    hp = torch.from_numpy(prompts).pin_memory()
    ht = torch.empty((P, G, T), dtype=torch.int32).pin_memory()
    hl = torch.empty((P, G, T), dtype=torch.float32).pin_memory()
    ver = eng.echo_rollout_host(hp, [Lp] * P, G, T, 1.0, 3, ht, hl)
    assert np.all(ver == 0)
    tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), [Lp] * P, G, T, 1.0, 3)
    eng.echo_sync()
    assert_same_rollout(ht.numpy(), hl.numpy(), tok.cpu().numpy(), lp.cpu().numpy())
    eng.close()


def _gpu_weights(w_t):
    return {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w_t.items()}


def _mean_abs_dlp(shape, w_o, prompts, lens, G, temp, seed, tok, lp, seqs):
    from helpers import score_sequences
    delta, _, _, _ = score_sequences(dims_of(shape), w_o, prompts, lens, G, temp, seed, tok, lp, seqs)
    return float(delta.mean())


@pytest.mark.parametrize("half_layers", [1, 2])
def test_half_operand_layers(B, tiny, half_layers):
    """echo_config.half_layers: the first layers keep their 16-bit operands in IEEE half.  Same
    acceptance rule against the (exact) oracle on every token, and the log-probabilities come out
    closer to it than with bf16 everywhere, scored along one common trajectory."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 3, 4, 24, 16
    prompts, lens = synth.make_ragged_prompts([24, 17, 9], wl.shape.vocab, 91, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=half_layers))
    eng.echo_load_policy(w_d, 1)
    tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 77)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 77, tok_h, lp_h, range(P * G))
    assert n == P * G * T and ex <= 0.05 * n
    eng.close()
    eng0 = B.Engine(B.make_config(wl.shape, P, G, Lp, T))
    eng0.echo_load_policy(w_d, 1)
    _, lp0, _ = eng0.echo_rollout(dp, lens, G, T, 1.0, 77, forced=tok)
    eng0.echo_sync()
    eng0.close()
    e_half = _mean_abs_dlp(wl.shape, w_o, prompts, lens, G, 1.0, 77, tok_h, lp_h, range(P * G))
    e_bf16 = _mean_abs_dlp(wl.shape, w_o, prompts, lens, G, 1.0, 77, tok_h, lp0.cpu().numpy(), range(P * G))
    assert e_half < 0.85 * e_bf16, (e_half, e_bf16)
    cfg = B.make_config(wl.shape, P, G, Lp, T)
    cfg.half_layers = wl.shape.n_layers + 1                      # more layers than the model has
    with pytest.raises(B.EchoError):
        B.Engine(cfg)


def test_rollout_past_the_suffix_kernel_switch(B):
    """A rollout of 1200 new tokens: from decode step 1088 on the engine replays its second captured
    graph (one suffix CTA per (sequence, kv head) instead of resident CTAs).  Two sequences are scored
    by the oracle on every step, before and after the switch; narrow and shallow enough (0.6B width,
    6 layers, 32000 ids) for the oracle to replay 1248 positions in seconds."""
    import dataclasses
    shape = dataclasses.replace(synth.SHAPES["0.6B"], name="0.6B-width L6", n_layers=6, vocab=32000)
    P, G, Lp, T = 4, 8, 48, 1200
    w_t = synth.make_weights(shape, 3, device="cuda")
    w_o = decoder.Weights(synth.weights_to_bits(w_t))
    eng = B.Engine(B.make_config(shape, P, G, Lp, T, 1))
    eng.echo_load_policy(w_t, 2)
    prompts = synth.make_prompts(P, Lp, shape.vocab, 17)
    lens = [Lp] * P
    tok, lp, ver = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 5)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    assert np.all(ver == 2) and eng.echo_get_stats()["decode_steps"] == T - 1
    n, ex, worst = check_sequences(dims_of(shape), w_o, prompts, lens, G, 1.0, 5, tok_h, lp_h, [6, 25])
    assert n == 2 * T and ex <= 0.03 * n
    # the same trajectory through the teacher-forced entry point (it crosses the switch too)
    _, lp_f, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 5, forced=tok)
    eng.echo_sync()
    assert np.max(np.abs(lp_f.cpu().numpy() - lp_h)) < LOGPROB_TOL
    eng.close()


def test_eight_query_heads_per_kv_head(B):
    """Hq / Hkv = 8 with G = 8 (the 32B shape's ratio): a group's 64 query rows take two prefix CTAs
    per (prompt, kv head) and the merge area of the resident suffix kernel is too small, so every
    step runs the per-item suffix kernel.  Every token of a small model against the oracle."""
    shape = synth.DecoderShape("rep8", 2, 512, 16, 2, 128, 1024, 4096)
    P, G, T = 3, 8, 24
    w_t = synth.make_weights(shape, 11)
    w_o = decoder.Weights(synth.weights_to_bits(w_t))
    prompts, lens = synth.make_ragged_prompts([40, 33, 17], shape.vocab, 23, pad_to=40)
    for hl in (0, 1):
        eng = B.Engine(B.make_config(shape, P, G, 40, T, 1, half_layers=hl))
        eng.echo_load_policy(_gpu_weights(w_t), 1)
        tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 99)
        eng.echo_sync()
        n, ex, worst = check_sequences(dims_of(shape), w_o, prompts, lens, G, 1.0, 99, tok.cpu().numpy(),
                                       lp.cpu().numpy(), range(P * G))
        assert n == P * G * T and ex <= 0.05 * n
        eng.close()


def test_every_sequence_ended_and_padded_trajectories(B, tiny, monkeypatch):
    """Teacher-forced scoring of trajectories that all end early and are padded with OTHER ids after
    their end token (a buffer from elsewhere): positions after the end token score the end token with
    log-probability 0 whatever the padding holds, with both suffix kernels (with one CTA per item,
    every CTA of the launch returns early once all sequences have ended).  The context then serves
    an ordinary rollout correctly."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 2, 4, 20, 10
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 41)
    lens = [Lp, Lp - 4]
    dp = torch.from_numpy(prompts).cuda()
    eos = 123
    rng = np.random.default_rng(3)
    given = rng.integers(0, wl.shape.vocab, size=(P, G, T)).astype(np.int32)
    given[given == eos] = eos + 1
    ends = rng.integers(0, 3, size=(P, G))                       # every sequence ends within three steps
    for p in range(P):
        for g in range(G):
            given[p, g, ends[p, g]] = eos                        # ... and what follows is NOT the end token
    for impl in ("", "waves"):
        if impl:
            monkeypatch.setenv("ECHO_ATTN_IMPL", impl)
        else:
            monkeypatch.delenv("ECHO_ATTN_IMPL", raising=False)
        eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, eos_id=eos))
        eng.echo_load_policy(w_d, 1)
        tok_f, lp_f, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 9, forced=torch.from_numpy(given).cuda())
        eng.echo_sync()
        tok_f, lp_f = tok_f.cpu().numpy(), lp_f.cpu().numpy()
        for p in range(P):
            for g in range(G):
                e = ends[p, g]
                assert np.all(lp_f[p, g, e + 1:] == 0.0) and np.all(tok_f[p, g, e + 1:] == eos)
                sc = decoder.score_forced(dims_of(wl.shape), w_o, prompts[p][: lens[p]], given[p, g], 1.0, 9,
                                          p * G + g, eos_id=eos)
                assert np.max(np.abs(lp_f[p, g] - sc.logprob_given)) <= LOGPROB_TOL
        tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 9)
        eng.echo_sync()
        check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 9, tok.cpu().numpy(), lp.cpu().numpy(),
                        range(P * G), eos_id=eos)
        eng.close()


def test_prompts_cut_over_contexts_reproduce_one_call(B, tiny):
    """Groups are independent: a prompt set cut by prompt over two contexts (as over two GPUs), each
    with its sequence-id base, yields the tokens one call over the whole set yields."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 4, 4, 32, 12
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 55)
    lens = [Lp] * P
    eng = _engine(B, wl.shape, P, G, Lp, T)
    eng.echo_load_policy(w_d, 1)
    tok_all, lp_all, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 321)
    eng.echo_sync()
    tok_all, lp_all = tok_all.cpu().numpy(), lp_all.cpu().numpy()
    n_parts = 2
    for r in range(n_parts):
        mine = [p for p in range(P) if p % n_parts == r]
        for p in mine:                        # one call per prompt here: its ids are p*G .. p*G+G-1
            eng.echo_set_sequence_base(p * G)
            tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts[p: p + 1]).cuda(), [Lp], G, T, 1.0, 321)
            eng.echo_sync()
            assert_same_rollout(tok.cpu().numpy()[0], lp.cpu().numpy()[0], tok_all[p], lp_all[p])
    eng.echo_set_sequence_base(0)
    eng.close()


@pytest.mark.parametrize("prefill", ["tiles", "rows"])
def test_prefill_attention_kernels(B, tiny, monkeypatch, prefill):
    """Prompt prefill with the tensor-core tile kernel (default) and with the one-query-per-row kernel
    (ECHO_ATTN_PREFILL=rows, also what serves page sizes other than 16): ragged prompts whose rows
    straddle prompt boundaries inside one CTA, lengths that are not multiples of the page size, a
    one-token prompt; every token against the oracle, with bf16 and with half operands."""
    wl, w_o, w_d = tiny
    if prefill == "rows":
        monkeypatch.setenv("ECHO_ATTN_PREFILL", "rows")
    else:
        monkeypatch.delenv("ECHO_ATTN_PREFILL", raising=False)
    lens_list = [37, 3, 1, 64, 18, 5, 33]
    P, G, Lp, T = len(lens_list), 2, 64, 6
    prompts, lens = synth.make_ragged_prompts(lens_list, wl.shape.vocab, 404, pad_to=Lp)
    for hl in (0, 2):
        eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=hl))
        eng.echo_load_policy(w_d, 1)
        tok, lp, _ = eng.echo_rollout(torch.from_numpy(prompts).cuda(), lens, G, T, 1.0, 808)
        eng.echo_sync()
        n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 808, tok.cpu().numpy(),
                                       lp.cpu().numpy(), range(P * G))
        assert n == P * G * T and ex <= 3
        eng.close()


def test_prefill_shaped_scoring(B, tiny):
    """echo_score: log-probabilities of given trajectories in prefill-shaped passes.  Against the oracle
    on every token (ragged prompts, lengths that are not multiples of the page size), against the
    decode-shaped teacher-forced entry point, with the end-of-sequence rule, and for T = 1."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 3, 4, 40, 14
    prompts, lens = synth.make_ragged_prompts([40, 21, 7], wl.shape.vocab, 515, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    for hl in (0, 2):
        eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=hl))
        eng.echo_load_policy(w_d, 4)
        tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 0.9, 11)
        lp_s, ver = eng.echo_score(dp, lens, tok, 0.9)
        _, lp_f, _ = eng.echo_rollout(dp, lens, G, T, 0.9, 11, forced=tok)
        eng.echo_sync()
        tok_h, lp_s, lp_f = tok.cpu().numpy(), lp_s.cpu().numpy(), lp_f.cpu().numpy()
        assert np.all(ver == 4) and np.all(lp_s <= 0)
        assert np.max(np.abs(lp_s - lp_f)) < LOGPROB_TOL / 5
        n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 0.9, 11, tok_h, lp_s, range(P * G))
        assert n == P * G * T
        # a single token per sequence: only the prompt pass and the first-token rows
        lp1, _ = eng.echo_score(dp, lens, tok[:, :, :1].contiguous(), 0.9)
        eng.echo_sync()
        assert np.max(np.abs(lp1.cpu().numpy()[..., 0] - lp_s[..., 0])) < LOGPROB_TOL / 5
        eng.close()
    # end-of-sequence rule: positions after a sequence's first end token score 0, the others are unchanged
    eos = int(tok_h[1, 2, 5])
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, eos_id=eos))
    eng.echo_load_policy(w_d, 1)
    lp_e, _ = eng.echo_score(dp, lens, tok, 0.9)
    eng.echo_sync()
    lp_e = lp_e.cpu().numpy()
    ended = np.zeros_like(tok_h, dtype=bool)
    ended[..., 1:] = np.logical_or.accumulate(tok_h[..., :-1] == eos, axis=-1)
    assert ended.any() and np.all(lp_e[ended] == 0.0)
    for s in range(P * G):
        p, g = divmod(s, G)
        sc = decoder.score_forced(dims_of(wl.shape), w_o, prompts[p][: lens[p]], tok_h[p, g], 0.9, 11, s, eos_id=eos)
        assert np.max(np.abs(lp_e[p, g] - sc.logprob_given)) <= LOGPROB_TOL
    eng.close()


def test_prefill_shaped_scoring_is_faster_than_stepwise(B):
    """A few hundred tokens per sequence at the 0.6B width: the scoring pass agrees with the decode-shaped
    teacher-forced entry point on every token and takes a fraction of its time."""
    import dataclasses
    shape = dataclasses.replace(synth.SHAPES["0.6B"], name="0.6B-width L6", n_layers=6, vocab=32000)
    P, G, Lp, T = 8, 8, 64, 384
    w_t = synth.make_weights(shape, 3, device="cuda")
    eng = B.Engine(B.make_config(shape, P, G, Lp, T, 1))
    eng.echo_load_policy(w_t, 1)
    prompts = torch.from_numpy(synth.make_prompts(P, Lp, shape.vocab, 29)).cuda()
    lens = [Lp] * P
    tok, lp, _ = eng.echo_rollout(prompts, lens, G, T, 1.0, 3)
    eng.echo_sync()
    times = {}
    for name in ("score", "forced"):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(eng.stream)
        if name == "score":
            lp_s, _ = eng.echo_score(prompts, lens, tok, 1.0)
        else:
            _, lp_f, _ = eng.echo_rollout(prompts, lens, G, T, 1.0, 3, forced=tok)
        e1.record(eng.stream)
        eng.echo_sync()
        times[name] = e0.elapsed_time(e1)
    d = (lp_s - lp_f).abs()
    print(f"score {times['score']:.1f} ms, stepwise {times['forced']:.1f} ms, max |dlogprob| {float(d.max()):.2e}")
    assert float(d.max()) < LOGPROB_TOL / 2 and float((lp_s - lp).abs().max()) < LOGPROB_TOL / 2
    assert times["score"] < 0.6 * times["forced"]
    eng.close()


def test_turn_mask_matches_oracle(B):
    from oracle import objective
    rng = np.random.default_rng(8)
    for n, T, p_start in [(1, 1, 0.5), (7, 33, 0.2), (64, 2048, 0.01), (300, 100, 0.0)]:
        x = rng.integers(0, 50, size=(n, T)).astype(np.int32)
        x[rng.random((n, T)) < p_start] = 77
        for shift in (False, True):
            got = B.echo_turn_mask(torch.from_numpy(x).cuda(), 77, shift).cpu().numpy()
            assert np.array_equal(got, objective.turn_mask(x, 77, shift))


def test_rollout_of_8192_new_tokens(B):
    """Section 5.1 generates up to 8192 new tokens per response.  A small two-layer model (head_dim 128,
    two query heads on one kv head) decodes 8192 tokens per sequence: 513 KV pages per sequence, the
    rotation table to position 8212, both captured graphs; one whole sequence is scored by the oracle
    (a causal pass over 8211 positions), every step, and the scoring entry point replays it."""
    shape = synth.DecoderShape("long", 2, 256, 2, 1, 128, 512, 2048)
    P, G, Lp, T = 1, 2, 20, 8192
    w_t = synth.make_weights(shape, 21)
    w_o = decoder.Weights(synth.weights_to_bits(w_t))
    eng = B.Engine(B.make_config(shape, P, G, Lp, T, 1))
    eng.echo_load_policy(_gpu_weights(w_t), 1)
    prompts = synth.make_prompts(P, Lp, shape.vocab, 61)
    dp = torch.from_numpy(prompts).cuda()
    tok, lp, _ = eng.echo_rollout(dp, [Lp], G, T, 1.0, 77)
    st = eng.echo_get_stats()
    assert st["decode_steps"] == T - 1 and st["n_pages"] == 2 + 2 * 513
    lp_s, _ = eng.echo_score(dp, [Lp], tok, 1.0)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    n, ex, worst = check_sequences(dims_of(shape), w_o, prompts, [Lp], G, 1.0, 77, tok_h, lp_h, [1])
    assert n == T and ex <= 0.03 * T
    assert float((lp_s - lp).abs().max()) < LOGPROB_TOL / 2
    eng.close()


def test_ended_sequences_leave_the_projection_rows(B, tiny, monkeypatch):
    """With an end token the decode steps run on the rows of the sequences that have not ended: they are
    packed to the front each step, and the host lowers the row count of the projections (64 -> 32 here)
    as the count of live sequences, which it follows two windows of steps behind the GPU, falls.
    Trajectories that end at scattered steps are scored teacher-forced: every position against the
    oracle, ended positions = end token / 0, and the same outputs as with the packing switched off."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 8, 8, 16, 200
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 606)
    lens = [Lp] * P
    dp = torch.from_numpy(prompts).cuda()
    eos = 7
    rng = np.random.default_rng(12)
    given = rng.integers(8, wl.shape.vocab, size=(P, G, T)).astype(np.int32)
    ends = rng.integers(0, 150, size=(P, G))
    ends[0, 0] = T + 5                                           # one sequence never ends
    ends[3, 2] = 0                                               # one ends with its first token
    for p in range(P):
        for g in range(G):
            if ends[p, g] < T:
                given[p, g, ends[p, g]] = eos
    forced = torch.from_numpy(given).cuda()
    out = {}
    for mode in ("packed", "unpacked"):
        if mode == "unpacked":
            monkeypatch.setenv("ECHO_NO_COMPACT", "1")
        else:
            monkeypatch.delenv("ECHO_NO_COMPACT", raising=False)
        eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, eos_id=eos))
        eng.echo_load_policy(w_d, 1)
        tok_f, lp_f, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 4, forced=forced)
        eng.echo_sync()
        out[mode] = (tok_f.cpu().numpy(), lp_f.cpu().numpy())
        # all but one sequence have ended by step 150: the last steps ran on 32 rows instead of 64
        assert eng.echo_get_stats()["last_step_rows"] == (32 if mode == "packed" else 64)
        # the context then serves a free-running rollout (all rows live again at its start)
        tok, lp, _ = eng.echo_rollout(dp, lens, G, 12, 1.0, 4)
        eng.echo_sync()
        check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 4, tok.cpu().numpy(), lp.cpu().numpy(),
                        [0, 19, 63], eos_id=eos)
        eng.close()
    tok_f, lp_f = out["packed"]
    for p in range(P):
        for g in range(G):
            e = ends[p, g]
            if e < T:
                assert np.all(lp_f[p, g, e + 1:] == 0.0) and np.all(tok_f[p, g, e + 1:] == eos)
    for s in (0, 1, 26, 40, 63):
        p, g = divmod(s, G)
        sc = decoder.score_forced(dims_of(wl.shape), w_o, prompts[p], given[p, g], 1.0, 4, s, eos_id=eos)
        assert np.max(np.abs(lp_f[p, g] - sc.logprob_given)) <= LOGPROB_TOL
        live = np.arange(T) <= min(ends[p, g], T - 1)
        diff = (tok_f[p, g] != sc.own_token) & live
        assert np.all(sc.margin[diff] < 1e-2) and np.all(tok_f[p, g][diff] == sc.runner_up[diff])
    assert np.max(np.abs(out["unpacked"][1] - lp_f)) < LOGPROB_TOL / 5
    assert (out["unpacked"][0] == tok_f).mean() > 0.99


@pytest.mark.parametrize("env", [{"ECHO_DETERMINISTIC": "1"}, {"ECHO_GEMM_IMPL": "single"}, {"ECHO_GEMM_IMPL": "simt"},
                                 {"ECHO_NO_GRAPH": "1"}, {"ECHO_NO_PDL": "1"}, {"ECHO_ATTN_IMPL": "rows"}])
def test_diagnostic_switches_keep_parity(B, tiny, monkeypatch, env):
    """The switches read at echo_create select other kernels or launch modes for the same arithmetic:
    fixed-order reductions (then two runs are bit-identical), the one-CTA and the plain projection
    kernels, no graph replay, no early kernel start, the general attention kernel.  Each against the
    oracle on every token, with half operands in the first layer and the end-of-sequence rule on."""
    wl, w_o, w_d = tiny
    for k in ("ECHO_DETERMINISTIC", "ECHO_GEMM_IMPL", "ECHO_NO_GRAPH", "ECHO_NO_PDL", "ECHO_ATTN_IMPL"):
        monkeypatch.delenv(k, raising=False)
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    P, G, Lp, T = 5, 8, 48, 40                      # 40 sequences: both projection kernel families see > 32 rows
    prompts, lens = synth.make_ragged_prompts([48, 31, 16, 5, 40], wl.shape.vocab, 313, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=1))
    eng.echo_load_policy(w_d, 1)
    tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 99)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    eng.close()
    eos = int(tok_h[2, 3, 7])
    eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=1, eos_id=eos))
    eng.echo_load_policy(w_d, 1)
    tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 99)
    tok2, lp2, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 99)
    eng.echo_sync()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 99, tok_h, lp_h, range(P * G),
                                   eos_id=eos)
    assert n == P * G * T and ex <= 0.05 * n
    assert np.any(tok_h[2, 3] == eos)
    if env.get("ECHO_DETERMINISTIC") == "1":
        assert np.array_equal(tok2.cpu().numpy(), tok_h) and np.array_equal(lp2.cpu().numpy(), lp_h)
    else:
        assert_same_rollout(tok2.cpu().numpy(), lp2.cpu().numpy(), tok_h, lp_h)
    eng.close()


def test_rmsnorm_as_projection_prologue(B, tiny, monkeypatch):
    """ECHO_FUSE_NORM=1 moves the two RMSNorms of a decode layer into the projections that consume them
    (a grid-wide barrier inside the kernel; needs more than 64 activation rows).  Same arithmetic: every
    token against the oracle, and the step holds two kernels per layer fewer."""
    wl, w_o, w_d = tiny
    P, G, Lp, T = 9, 8, 24, 12
    prompts, lens = synth.make_ragged_prompts([24, 9, 17, 24, 3, 20, 11, 24, 6], wl.shape.vocab, 77, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    launched = {}
    for mode in ("0", "1"):
        monkeypatch.setenv("ECHO_FUSE_NORM", mode)
        eng = B.Engine(B.make_config(wl.shape, P, G, Lp, T, half_layers=1))
        eng.echo_load_policy(w_d, 1)
        tok, lp, _ = eng.echo_rollout(dp, lens, G, T, 1.0, 5)
        eng.echo_sync()
        launched[mode] = eng.echo_get_stats()["kernels_launched"]
        n, ex, worst = check_sequences(dims_of(wl.shape), w_o, prompts, lens, G, 1.0, 5, tok.cpu().numpy(),
                                       lp.cpu().numpy(), range(0, P * G, 5))
        assert ex <= 0.05 * n
        eng.close()
    assert launched["0"] - launched["1"] == 2 * wl.shape.n_layers * (T - 1)


def test_prompt_queue_refills_freed_slots(B, tiny):
    """echo_rollout_queue: 11 prompts through a context of 6 group slots.  A slot is refilled from the queue
    when all of its samples have ended, between two decode steps of the others.  Every sequence keeps the
    noise stream of its id and counts its tokens from its own admission, so every token of every sequence
    is checked against the oracle's rollout of that sequence alone, and against one echo_rollout call of a
    context that holds all 11 prompts at once.  Free-running without an end token (slots turn over by
    length: two waves), then teacher-forced along given tokens that end at very different lengths."""
    wl, w_o, w_d = tiny
    Pq, S, G, Lp, T = 11, 6, 8, 40, 56
    prompts, lens = synth.make_ragged_prompts([40, 7, 33, 16, 40, 1, 25, 17, 32, 9, 21], wl.shape.vocab, 909, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    dims = dims_of(wl.shape)
    # ---- no end token ---------------------------------------------------------------------------
    big = B.Engine(B.make_config(wl.shape, Pq, G, Lp, T))
    big.echo_load_policy(w_d, 3)
    tok_all, lp_all, _ = big.echo_rollout(dp, lens, G, T, 1.0, 4242)
    big.echo_sync()
    tok_all, lp_all = tok_all.cpu().numpy(), lp_all.cpu().numpy()
    big.close()
    eng = B.Engine(B.make_config(wl.shape, S, G, Lp, T))
    eng.echo_load_policy(w_d, 3)
    tok, lp, ver = eng.echo_rollout_queue(dp, lens, G, T, 1.0, 4242)
    eng.echo_sync()
    st = eng.echo_get_stats()
    tok_h, lp_h = tok.cpu().numpy(), lp.cpu().numpy()
    assert tok_h.shape == (Pq, G, T) and np.all(ver == 3) and st["tokens_generated"] == Pq * G * T
    assert st["decode_steps"] == 2 * (T - 1)
    n, ex, worst = check_sequences(dims, w_o, prompts, lens, G, 1.0, 4242, tok_h, lp_h, range(Pq * G))
    assert n == Pq * G * T and ex <= 0.05 * n
    assert_same_rollout(tok_h, lp_h, tok_all, lp_all)
    # a second call on the same context (slots, flags and tables start over); fewer prompts than slots;
    # a single new token per sequence (no decode step at all)
    tok2, lp2, _ = eng.echo_rollout_queue(dp, lens, G, T, 1.0, 4242)
    tok3, lp3, _ = eng.echo_rollout_queue(dp[:2].contiguous(), lens[:2], G, T, 1.0, 4242)
    tok4, lp4, _ = eng.echo_rollout_queue(dp, lens, G, 1, 1.0, 4242)
    eng.echo_sync()
    assert_same_rollout(tok2.cpu().numpy(), lp2.cpu().numpy(), tok_h, lp_h)
    assert_same_rollout(tok3.cpu().numpy(), lp3.cpu().numpy(), tok_h[:2], lp_h[:2])
    assert_same_rollout(tok4.cpu().numpy(), lp4.cpu().numpy(), tok_h[:, :, :1], lp_h[:, :, :1])
    eng.close()
    # ---- given tokens with an end token at a random place --------------------------------------------
    eos = 7
    rng = np.random.default_rng(5)
    given = rng.integers(8, wl.shape.vocab, size=(Pq, G, T)).astype(np.int32)
    ends = rng.integers(0, 30, size=(Pq, G))
    ends[4] = rng.integers(0, 6, size=G)                         # one group ends at once: its slot turns over early
    ends[0, 0] = T + 5                                           # one sequence never ends
    for p in range(Pq):
        for g in range(G):
            if ends[p, g] < T:
                given[p, g, ends[p, g]] = eos
    forced = torch.from_numpy(given).cuda()
    eng = B.Engine(B.make_config(wl.shape, S, G, Lp, T, eos_id=eos))
    eng.echo_load_policy(w_d, 3)
    tok_f, lp_f, _ = eng.echo_rollout_queue(dp, lens, G, T, 1.0, 4242, forced=forced)
    eng.echo_sync()
    st = eng.echo_get_stats()
    tok_f, lp_f = tok_f.cpu().numpy(), lp_f.cpu().numpy()
    assert T - 1 <= st["decode_steps"] < 2 * (T - 1) - 16        # fewer steps than two waves of six groups
    assert st["last_step_rows"] == 32                            # and the last ones on the smallest row count
    for s in range(Pq * G):
        p, g = divmod(s, G)
        e = ends[p, g]
        if e < T:
            assert np.all(lp_f[p, g, e + 1:] == 0.0) and np.all(tok_f[p, g, e + 1:] == eos)
        sc = decoder.score_forced(dims, w_o, prompts[p][: int(lens[p])], given[p, g], 1.0, 4242, s, eos_id=eos)
        assert np.max(np.abs(lp_f[p, g] - sc.logprob_given)) <= LOGPROB_TOL
        live = np.arange(T) <= min(e, T - 1)
        diff = (tok_f[p, g] != sc.own_token) & live
        assert np.all(sc.margin[diff] < 1e-2) and np.all(tok_f[p, g][diff] == sc.runner_up[diff])
    # the context then serves an ordinary rollout
    tok5, lp5, _ = eng.echo_rollout(dp[:S].contiguous(), lens[:S], G, 12, 1.0, 4242)
    eng.echo_sync()
    check_sequences(dims, w_o, prompts, lens, G, 1.0, 4242, tok5.cpu().numpy(), lp5.cpu().numpy(), range(S * G), eos_id=eos)
    eng.close()


def test_prompt_queue_with_a_small_page_pool(B, tiny):
    """More group slots than the KV pool could hold at full length: the queue hands a sequence its pages at
    admission and takes them back when the host has seen it ended, and admits by free pages and by the
    number of live sequences.  Same per-sequence check as above; the pool's peak stays within its size."""
    wl, w_o, w_d = tiny
    Pq, G, Lp, T = 14, 8, 40, 56
    lens_l = [40, 7, 33, 16, 40, 1, 25, 17, 32, 9, 21, 40, 3, 28]
    prompts, lens = synth.make_ragged_prompts(lens_l, wl.shape.vocab, 910, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    dims = dims_of(wl.shape)
    eos = 7
    rng = np.random.default_rng(6)
    given = rng.integers(8, wl.shape.vocab, size=(Pq, G, T)).astype(np.int32)
    ends = rng.integers(0, 40, size=(Pq, G))
    ends[1, 0] = T + 5
    for p in range(Pq):
        for g in range(G):
            if ends[p, g] < T:
                given[p, g, ends[p, g]] = eos
    forced = torch.from_numpy(given).cuda()
    Z = 16
    per_group = -(-Lp // Z) + G * (-(-(Lp % Z + T - 1) // Z))   # pages of one group at the longest prompt
    pool = 3 * per_group + 5                                      # three groups at full length and a little more
    eng = B.Engine(B.make_config(wl.shape, Pq, G, Lp, T, eos_id=eos, kv_pages=pool, queue_max_live=40))
    eng.echo_load_policy(w_d, 3)
    tok_f, lp_f, _ = eng.echo_rollout_queue(dp, lens, G, T, 1.0, 77, forced=forced)
    eng.echo_sync()
    st = eng.echo_get_stats()
    tok_f, lp_f = tok_f.cpu().numpy(), lp_f.cpu().numpy()
    assert 0 < st["n_pages"] <= pool
    for s in range(Pq * G):
        p, g = divmod(s, G)
        e = ends[p, g]
        if e < T:
            assert np.all(lp_f[p, g, e + 1:] == 0.0) and np.all(tok_f[p, g, e + 1:] == eos)
        sc = decoder.score_forced(dims, w_o, prompts[p][: int(lens[p])], given[p, g], 1.0, 77, s, eos_id=eos)
        assert np.max(np.abs(lp_f[p, g] - sc.logprob_given)) <= LOGPROB_TOL
        live = np.arange(T) <= min(e, T - 1)
        diff = (tok_f[p, g] != sc.own_token) & live
        assert np.all(sc.margin[diff] < 1e-2) and np.all(tok_f[p, g][diff] == sc.runner_up[diff])
    # free-running on the same context: sequences end only by length, groups pass through the pool three at a time
    tok, lp, _ = eng.echo_rollout_queue(dp, lens, G, 20, 1.0, 78)
    eng.echo_sync()
    check_sequences(dims, w_o, prompts, lens, G, 1.0, 78, tok.cpu().numpy(), lp.cpu().numpy(), range(0, Pq * G, 3),
                    eos_id=eos)
    eng.close()
    # the same with nucleus sampling and half operands in the first layer (the admission path samples token 0
    # of every admitted group through the same cut kernel as a decode step)
    eng = B.Engine(B.make_config(wl.shape, Pq, G, Lp, T, eos_id=eos, kv_pages=pool, queue_max_live=40, top_p=0.9,
                                 half_layers=1))
    eng.echo_load_policy(w_d, 3)
    tok, lp, _ = eng.echo_rollout_queue(dp, lens, G, 20, 1.0, 79)
    eng.echo_sync()
    n, ex, _ = check_sequences(dims, w_o, prompts, lens, G, 1.0, 79, tok.cpu().numpy(), lp.cpu().numpy(),
                               range(0, Pq * G, 3), eos_id=eos, top_p=0.9)
    assert ex <= 0.05 * n
    # a plain rollout of all 14 groups does not fit this pool and is refused; three groups do
    with pytest.raises(B.EchoError):
        eng.echo_rollout(dp, lens, G, T, 1.0, 78)
    tok5, lp5, _ = eng.echo_rollout(dp[:3].contiguous(), lens[:3], G, 12, 1.0, 78)
    eng.echo_sync()
    check_sequences(dims, w_o, prompts, lens, G, 1.0, 78, tok5.cpu().numpy(), lp5.cpu().numpy(), range(3 * G), eos_id=eos,
                    top_p=0.9)
    eng.close()


def test_snapshot_from_a_chain_buffer_installs_and_serves(B, tiny):
    """What a forwarding chain delivers is one flat byte buffer in this GPU's memory (chain.pack on the
    sender, chunked transfers, chain.unpack on the receiver: views, no copy).  Installed from those views,
    in chunks that arrive while the previous version is serving, it must serve exactly the rollout that a
    direct install of the same snapshot serves, and the oracle's."""
    from paper_2602_02192_b200 import chain
    wl, w_o, w_d = tiny
    w1_t = synth.make_weights(wl.shape, 21)
    w1_o = decoder.Weights(synth.weights_to_bits(w1_t))
    flat_src = chain.pack(w1_t, wl.shape)                               # on the sending side (host memory here)
    entries, total = chain.snapshot_layout(wl.shape)
    assert flat_src.numel() == total and all(off % 256 == 0 for _, _, off, _ in entries)
    P, G, Lp, T = 3, 4, 16, 10
    prompts = synth.make_prompts(P, Lp, wl.shape.vocab, 8)
    dp = torch.from_numpy(prompts).cuda()
    eng = _engine(B, wl.shape, P, G, Lp, T)
    eng.echo_load_policy(w_d, 1)
    t0, _, v0 = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 5)            # version 1 serves ...
    flat = torch.empty(total, dtype=torch.uint8, device="cuda")          # ... while the chunks land
    chunk = 1 << 16
    for a in range(0, total, chunk):
        flat[a:a + chunk].copy_(flat_src[a:a + chunk], non_blocking=True)
    torch.cuda.current_stream().synchronize()
    eng.echo_load_policy(chain.unpack(flat, wl.shape), 2)
    eng.echo_wait_policy()
    t1, l1, v1 = eng.echo_rollout(dp, [Lp] * P, G, T, 1.0, 5)
    eng.echo_sync()
    assert np.all(v0 == 1) and np.all(v1 == 2)
    check_sequences(dims_of(wl.shape), w1_o, prompts, [Lp] * P, G, 1.0, 5, t1.cpu().numpy(), l1.cpu().numpy(),
                    range(P * G))
    eng.close()
    ref = _engine(B, wl.shape, P, G, Lp, T)
    ref.echo_load_policy({k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w1_t.items()}, 2)
    t2, l2, _ = ref.echo_rollout(dp, [Lp] * P, G, T, 1.0, 5)
    ref.echo_sync()
    assert_same_rollout(t2.cpu().numpy(), l2.cpu().numpy(), t1.cpu().numpy(), l1.cpu().numpy())
    ref.close()


def test_prompt_queue_optimistic_pages_and_eviction(B, tiny):
    """queue_optimistic: pages are handed out window by window, groups are admitted without room for their
    longest continuation, and when the pool cannot cover the next window the newest groups are evicted and
    generated again later.  An evicted group's second run gives the same tokens (noise keyed by sequence id
    and token index), so every sequence still matches the oracle's rollout of that sequence alone; the run
    needs fewer decode steps than the one that reserves every continuation, in the same pool."""
    wl, w_o, w_d = tiny
    Pq, G, Lp, T = 14, 8, 40, 56
    lens_l = [40, 7, 33, 16, 40, 1, 25, 17, 32, 9, 21, 40, 3, 28]
    prompts, lens = synth.make_ragged_prompts(lens_l, wl.shape.vocab, 910, pad_to=Lp)
    dp = torch.from_numpy(prompts).cuda()
    dims = dims_of(wl.shape)
    eos = 7
    rng = np.random.default_rng(6)
    given = rng.integers(8, wl.shape.vocab, size=(Pq, G, T)).astype(np.int32)
    ends = rng.integers(0, T + 10, size=(Pq, G))
    for p in range(Pq):
        for g in range(G):
            if ends[p, g] < T:
                given[p, g, ends[p, g]] = eos
    forced = torch.from_numpy(given).cuda()
    stats = {}
    for mode in (0, 1):
        eng = B.Engine(B.make_config(wl.shape, Pq, G, Lp, T, eos_id=eos, kv_pages=60, queue_optimistic=mode))
        eng.echo_load_policy(w_d, 3)
        tok_f, lp_f, _ = eng.echo_rollout_queue(dp, lens, G, T, 1.0, 77, forced=forced)
        eng.echo_sync()
        stats[mode] = eng.echo_get_stats()
        tok_f, lp_f = tok_f.cpu().numpy(), lp_f.cpu().numpy()
        assert 0 < stats[mode]["n_pages"] <= 60
        for s in range(Pq * G):
            p, g = divmod(s, G)
            e = ends[p, g]
            if e < T:
                assert np.all(lp_f[p, g, e + 1:] == 0.0) and np.all(tok_f[p, g, e + 1:] == eos)
            sc = decoder.score_forced(dims, w_o, prompts[p][: int(lens[p])], given[p, g], 1.0, 77, s, eos_id=eos)
            assert np.max(np.abs(lp_f[p, g] - sc.logprob_given)) <= LOGPROB_TOL
            live = np.arange(T) <= min(e, T - 1)
            diff = (tok_f[p, g] != sc.own_token) & live
            assert np.all(sc.margin[diff] < 1e-2) and np.all(tok_f[p, g][diff] == sc.runner_up[diff])
        if mode == 1:
            # free-running too (no sequence ends early: the pool is under the most pressure)
            tok, lp, _ = eng.echo_rollout_queue(dp, lens, G, 24, 1.0, 78)
            eng.echo_sync()
            assert eng.echo_get_stats()["queue_evictions"] > 0
            check_sequences(dims, w_o, prompts, lens, G, 1.0, 78, tok.cpu().numpy(), lp.cpu().numpy(),
                            range(0, Pq * G, 3), eos_id=eos)
        eng.close()
    assert stats[0]["queue_evictions"] == 0 and stats[1]["queue_evictions"] > 0
    assert stats[1]["decode_steps"] < stats[0]["decode_steps"]
