"""GPU parity of the stand-alone kernels against the CPU oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

from oracle import advantage as o_adv
from oracle import philox as o_philox
from oracle import sampler as o_sampler
from oracle.decoder import widen_bf16
from paper_2602_02192_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_02192_b200 import binding
    return binding


def test_noise_words_and_uniforms_bit_exact(B):
    total = 0
    rng = np.random.default_rng(0)
    for _ in range(8):
        seed = int(rng.integers(0, 1 << 63)) * 2 + int(rng.integers(0, 2))
        s, j = int(rng.integers(0, 1 << 20)), int(rng.integers(0, 1 << 13))
        V = 151936
        words, uni = B.echo_debug_noise(seed, s, j, 0, V)
        torch.cuda.synchronize()
        want_w = o_philox.noise_words(seed, s, j, V)
        assert np.array_equal(words.cpu().numpy().view(np.uint32), want_w)
        want_u = o_philox.uniform_from_word(want_w)
        assert np.array_equal(uni.cpu().numpy().view(np.uint32), want_u.view(np.uint32))
        total += V
    # ragged start / length
    words, uni = B.echo_debug_noise(5, 3, 2, 1001, 77)
    assert np.array_equal(words.cpu().numpy().view(np.uint32), o_philox.noise_words(5, 3, 2, 1001 + 77)[1001:])
    assert total > 1_000_000


@pytest.mark.parametrize("V,R,G,temp", [(4096, 16, 4, 1.0), (151936, 6, 2, 1.0), (1003, 5, 1, 0.7), (7, 3, 3, 1.5)])
def test_sampler_matches_oracle(B, V, R, G, temp):
    rng = np.random.default_rng(V)
    n_rows = (R + G - 1) // G
    z = (rng.normal(size=(n_rows, V)) * 1.3).astype(np.float32)
    seed, j = 0x1234567_89ABCDEF, 3
    tok, lp = B.echo_sample(torch.from_numpy(z).cuda(), R, G, j, temp, seed)
    forced = torch.from_numpy(rng.integers(0, V, size=R).astype(np.int32)).cuda()
    tok_f, lp_f = B.echo_sample(torch.from_numpy(z).cuda(), R, G, j, temp, seed, forced=forced)
    tok, lp, tok_f, lp_f = tok.cpu().numpy(), lp.cpu().numpy(), tok_f.cpu().numpy(), lp_f.cpu().numpy()
    for r in range(R):
        d = o_sampler.draw(z[r // G], temp, seed, r, j)
        if tok[r] != d.token:
            assert d.margin < 1e-4 and tok[r] == d.runner_up
        assert abs(lp[r] - d.logprobs[tok[r]]) < 2e-5 * max(1.0, abs(d.logprobs[tok[r]]))
        assert tok_f[r] == tok[r]
        assert abs(lp_f[r] - d.logprobs[int(forced[r])]) < 2e-5 * max(1.0, abs(d.logprobs[int(forced[r])]))


def _row(kind, V, rng):
    if kind == "normal":
        return (rng.normal(size=V) * 1.3).astype(np.float32)
    if kind == "peaked":
        z = (rng.normal(size=V) * 0.5).astype(np.float32)
        z[rng.integers(0, V, size=5)] += np.float32(9.0)
        return z
    if kind == "equal":
        return np.full(V, 0.25, dtype=np.float32)
    if kind == "levels":                               # many exactly equal scores on a few levels
        return (np.round(rng.normal(size=V) * 2.0) / 2.0).astype(np.float32)
    raise ValueError(kind)


@pytest.mark.parametrize("V,kind,top_p,temp", [(8, "normal", 0.9, 1.0), (1000, "normal", 0.5, 0.7),
                                               (4096, "peaked", 0.95, 1.0), (151936, "normal", 0.95, 1.0),
                                               (151936, "equal", 0.95, 1.0), (151936, "levels", 0.9, 1.0),
                                               (50000, "levels", 0.3, 1.3), (151936, "peaked", 0.05, 1.0),
                                               (4096, "normal", 1.0, 1.0)])
def test_top_p_sampler_matches_oracle(B, V, kind, top_p, temp):
    """Nucleus cut, draw and renormalised log-probability against the oracle.  The cut is found from
    fp32 mass sums, so it may sit a few ids away from the oracle's fp64 one: the kernel's nucleus must
    be a prefix of the ranking whose mass reaches top_p and is minimal, both within 3e-5 of mass."""
    rng = np.random.default_rng(V + int(top_p * 1000))
    R = 6
    z = np.stack([_row(kind, V, rng) for _ in range(R)])
    seed, j = 0xABCDEF0123, 2
    zc = torch.from_numpy(z).cuda()
    tok, lp, cuts = B.echo_sample_top_p(zc, R, 1, j, temp, top_p, seed)
    forced = torch.from_numpy(rng.integers(0, V, size=R).astype(np.int32)).cuda()
    tok_f, lp_f, _ = B.echo_sample_top_p(zc, R, 1, j, temp, top_p, seed, forced=forced)
    tok, lp, tok_f, lp_f = tok.cpu().numpy(), lp.cpu().numpy(), tok_f.cpu().numpy(), lp_f.cpu().numpy()
    cuts = cuts.cpu().numpy().view(np.uint32)
    inv_t = np.float32(1.0) / np.float32(temp)
    ids = np.arange(V)
    for r in range(R):
        d = o_sampler.draw(z[r], temp, seed, r, j, top_p)
        lp_full = o_sampler.log_softmax(z[r].astype(np.float64) / temp)
        p = np.exp(lp_full)
        if top_p >= 1.0:
            mask = np.ones(V, dtype=bool)
        else:
            s32 = z[r] * inv_t                                   # the kernel's scores
            u = s32.view(np.uint32)
            key = np.where(u & 0x80000000, ~u, u | 0x80000000).astype(np.uint64)
            ck, cid = int(cuts[r, 0]), int(cuts[r, 1])
            mask = (key > ck) | ((key == ck) & (ids <= cid))
            order = np.lexsort((ids, -s32.astype(np.float64)))
            k = int(mask.sum())
            assert k >= 1 and np.all(mask[order[:k]])            # a prefix of the ranking
            mass = p[mask].sum()
            assert mass >= top_p - 3e-5                          # reaches the target ...
            assert mass - p[order[k - 1]] < top_p + 3e-5         # ... and no shorter prefix does
            assert abs(k - d.nucleus_size) <= 8                  # a few ids around the oracle's cut
        mass = p[mask].sum()
        assert mask[tok[r]]
        if tok[r] != d.token:
            both = mask & np.isfinite(d.logprobs)
            assert (d.margin < 1e-4 and tok[r] == d.runner_up) or not both[d.token] or not both[tok[r]]
        want = lp_full[tok[r]] - np.log(mass)
        assert abs(lp[r] - want) < 3e-5 * max(1.0, abs(want))
        if np.isfinite(d.logprobs[tok[r]]):
            assert abs(lp[r] - d.logprobs[tok[r]]) < 1e-4
        assert tok_f[r] == tok[r]
        f = int(forced[r])
        if mask[f]:
            wf = lp_full[f] - np.log(mass)
            assert abs(lp_f[r] - wf) < 3e-5 * max(1.0, abs(wf))
        else:
            assert np.isneginf(lp_f[r])


def test_sampler_seq_ids_and_tie_rule(B):
    V = 64
    z = np.zeros((1, V), dtype=np.float32)
    ids = torch.tensor([7, 3, 7], dtype=torch.int32).cuda()
    tok, _ = B.echo_sample(torch.from_numpy(z).cuda(), 3, 3, 0, 1.0, 99, seq_ids=ids)
    tok = tok.cpu().numpy()
    assert tok[0] == tok[2] == o_sampler.draw(z[0], 1.0, 99, 7, 0).token
    assert tok[1] == o_sampler.draw(z[0], 1.0, 99, 3, 0).token
    # huge equal logits on two ids swamp the noise only if it is equal too; instead check the
    # documented rule on a row where one id dominates by far: always that id
    z2 = np.full((1, V), -50.0, dtype=np.float32); z2[0, 11] = 50.0
    tok, lp = B.echo_sample(torch.from_numpy(z2).cuda(), 4, 4, 1, 1.0, 5)
    assert np.all(tok.cpu().numpy() == 11) and np.all(np.abs(lp.cpu().numpy()) < 1e-6)


@pytest.mark.parametrize("M,N,K", [(256, 384, 256), (16, 256, 256), (1, 128, 64), (100, 688, 256),
                                   (37, 256, 688), (300, 1024, 512), (256, 4096, 4096), (512, 640, 1024),
                                   (256, 4096, 12288), (130, 151936, 256), (300, 40000, 512), (100, 20000, 320)])
def test_gemm_tensor_core_matches_fp64(B, M, N, K):
    rng = np.random.default_rng(M * 1000003 + N * 101 + K)
    X = torch.from_numpy(rng.normal(size=(M, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy((rng.normal(size=(N, K)) * 0.05).astype(np.float32)).to(torch.bfloat16)
    want = widen_bf16(synth.bf16_bits(X)) @ widen_bf16(synth.bf16_bits(W)).T
    # fp32 accumulation of K products of magnitude ~0.05: error ~ K * 2^-24 * |terms|
    tol = 2e-6 * K * 0.05 * 4 + 1e-6
    # 1 = SIMT reference, 0 = automatic choice, 2 = persistent stream-K, 100+s = cluster split-K by s
    # 200+s = independent k-slices added into the output in memory (s = 0: automatic)
    # 300+s = SM-pair kernel (more than 64 rows) with s k-slices; +1000 = weights in the block-tiled layout
    impls = (1, 0, 2, 101, 103, 108, 200, 206, 1001, 1000, 1002, 1104, 1203) if N * K <= 4096 * 4096 else (0, 2, 200, 1000)
    if M > 64:
        impls += (300, 301, 303, 1300, 1302)
    else:
        with pytest.raises(B.EchoError):
            B.echo_gemm_bf16(X.cuda(), W.cuda(), impl=300)
    for impl in impls:
        Y = B.echo_gemm_bf16(X.cuda(), W.cuda(), impl=impl)
        got = Y.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - want)) < tol, (impl, np.max(np.abs(got - want)))
    # residual-add epilogue, twice in a row (the tile counters must return to zero)
    Y0 = torch.from_numpy(rng.normal(size=(M, N)).astype(np.float32)).cuda()
    Y = Y0.clone()
    B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=1, Y=Y, impl=2)
    B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=1, Y=Y, impl=200)
    got = Y.cpu().numpy().astype(np.float64)
    assert np.max(np.abs(got - (Y0.cpu().numpy() + 2 * want))) < 2 * tol + 1e-5
    if M > 64:
        Y = Y0.clone()
        B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=1, Y=Y, impl=300)
        B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=1, Y=Y, impl=1300)
        got = Y.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - (Y0.cpu().numpy() + 2 * want))) < 2 * tol + 1e-5


@pytest.mark.parametrize("M,F,K", [(256, 688, 256), (16, 64, 64), (77, 1000, 512), (256, 12288, 4096),
                                   (512, 3072, 1024)])
def test_gemm_swiglu_epilogue(B, M, F, K):
    rng = np.random.default_rng(M + F + K)
    X = torch.from_numpy(rng.normal(size=(M, K)).astype(np.float32)).to(torch.bfloat16)
    W = torch.from_numpy((rng.normal(size=(2 * F, K)) * 0.05).astype(np.float32)).to(torch.bfloat16)
    xf, wf = widen_bf16(synth.bf16_bits(X)), widen_bf16(synth.bf16_bits(W))
    g, u = xf @ wf[:F].T, xf @ wf[F:].T
    want = g / (1 + np.exp(-g)) * u
    for impl in (0, 2, 101, 104, 1000, 1002) + ((300, 1300) if M > 64 else ()):
        Y = B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=2, impl=impl)
        got = Y.float().cpu().numpy().astype(np.float64)
        # the output is rounded to bf16 (relative 2^-9) on top of the fp32 accumulation error
        assert np.all(np.abs(got - want) <= 2.0 ** -8 * np.abs(want) + 1e-4 * K / 256), impl
        Y2 = B.echo_gemm_bf16(X.cuda(), W.cuda(), epilogue=2, impl=impl)
        assert torch.equal(Y, Y2)                          # deterministic reduction order


@pytest.mark.parametrize("P,G,Hq,Hkv,hd,Lp,steps", [(4, 8, 32, 8, 128, 512, 1200), (3, 4, 4, 2, 64, 40, 37),
                                                     (2, 2, 16, 2, 128, 7, 1), (2, 8, 8, 8, 128, 64, 300),
                                                     (16, 8, 32, 8, 128, 64, 70), (20, 8, 16, 8, 128, 16, 2),
                                                     (40, 8, 8, 4, 64, 33, 150), (16, 8, 32, 8, 128, 512, 400),
                                                     (3, 8, 8, 2, 64, 48, 20), (2, 6, 32, 8, 128, 100, 9),
                                                     (2, 8, 16, 2, 128, 64, 30), (2, 5, 16, 2, 128, 80, 3)])
@pytest.mark.parametrize("fmt", ["bf16", "half"])
@pytest.mark.parametrize("suffix", ["resident", "waves", "tiles"])
def test_decode_attention_matches_oracle(B, suffix, fmt, P, G, Hq, Hkv, hd, Lp, steps):
    """Shared-prefix decode attention against the oracle's single-query attention (fp64) on the same
    16-bit q, K, V (bf16, or IEEE half as in the layers of echo_config.half_layers), gathered through
    the oracle's page plan.  Both suffix kernels (resident CTAs that walk several (sequence, kv head)
    items; "waves" = one CTA per item) and both prefix kernels (a group's query rows in one CTA where
    they fill two 16-row tiles; "tiles" = one CTA per tile)."""
    from oracle import decoder as o_dec
    from oracle import pages as o_pages
    rng = np.random.default_rng(P * 131 + Lp)
    plan = o_pages.build([Lp] * P, G, steps + 1, 16)
    n_pages, Bq = plan.n_pages, P * G
    dt = torch.bfloat16 if fmt == "bf16" else torch.float16
    pool = torch.from_numpy(rng.normal(size=(n_pages, Hkv, 2, 16, hd)).astype(np.float32)).to(dt)
    q = torch.from_numpy(rng.normal(size=(Bq, Hq, hd)).astype(np.float32)).to(dt)
    pos = np.full(Bq, Lp + steps - 1, dtype=np.int32)
    pos[::3] -= min(steps - 1, 5)                       # sequences need not be at the same position
    full = np.repeat(plan.full_prefix_pages, G).astype(np.int32)
    out = B.echo_decode_attention(q.cuda(), pool.cuda(), torch.from_numpy(plan.table).cuda(),
                                  torch.from_numpy(pos).cuda(), torch.from_numpy(full).cuda(), P, G,
                                  kernel_choice={"resident": 0, "waves": 1, "tiles": 2}[suffix])
    assert out.dtype == dt
    out = out.float().cpu().numpy().astype(np.float64)
    poolf = pool.to(torch.float64).numpy()                # exact widening of the 16-bit values
    qf = q.to(torch.float64).numpy()
    # more (sequence, kv head) items than CTAs fit the GPU at once: a resident CTA then walks several
    # items and prefetches across their boundaries, so every fifth sequence is checked
    many = Bq * Hkv > 400
    # probabilities and the output are rounded to the operand format: 2^-9 relative each for bf16,
    # 2^-12 for half (where the fp32 exponentials and sums show instead)
    rel, floor = (1.5e-2, 4e-3) if fmt == "bf16" else (2.5e-3, 6e-4)
    for s in sorted(set([0, 1, Bq // 2, Bq - 1] + (list(range(0, Bq, 5)) if many else []))):
        n = int(pos[s]) + 1
        pg = plan.table[s, np.arange(n) // 16]
        K = poolf[pg, :, 0, np.arange(n) % 16, :]         # [n, Hkv, hd]
        V = poolf[pg, :, 1, np.arange(n) % 16, :]
        want = o_dec.attend_one(qf[s], K, V, Hq, Hkv)
        err = np.abs(out[s] - want)
        assert np.all(err <= rel * np.abs(want) + floor), (s, err.max())


@pytest.mark.parametrize("M,N,K", [(256, 4096, 4096), (256, 6144, 1024), (100, 688, 256), (32, 512, 2048),
                                   (130, 20000, 320)])
def test_gemm_half_operands_match_fp64(B, M, N, K):
    """The projections of the layers configured with IEEE-half operands: same kernels, operand format
    half.  Against the fp64 product of the exactly widened inputs, all kernel families."""
    rng = np.random.default_rng(M + 7 * N + 13 * K)
    X = torch.from_numpy(rng.normal(size=(M, K)).astype(np.float32)).to(torch.float16)
    W = torch.from_numpy((rng.normal(size=(N, K)) * 0.05).astype(np.float32)).to(torch.float16)
    xf, wf = X.to(torch.float64).numpy(), W.to(torch.float64).numpy()
    want = xf @ wf.T
    tol = 2e-6 * K * 0.05 * 4 + 1e-6
    impls = (1, 0, 2, 102, 200, 1000, 1002) + ((300, 1300, 1302) if M > 64 else ())
    for impl in impls:
        got = B.echo_gemm_bf16(X.cuda(), W.cuda(), impl=impl).cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - want)) < tol, (impl, np.max(np.abs(got - want)))
    # SwiGLU epilogue with a half output (2^-11 relative)
    F = N // 2
    g, u = want[:, :F], want[:, F: 2 * F]
    act = g / (1 + np.exp(-g)) * u
    for impl in (0, 2, 1000) + ((300, 1300) if M > 64 else ()):
        Y = B.echo_gemm_bf16(X.cuda(), W[: 2 * F].contiguous().cuda(), epilogue=2, impl=impl)
        assert Y.dtype == torch.float16
        got = Y.to(torch.float64).cpu().numpy()
        assert np.all(np.abs(got - act) <= 2.0 ** -10 * np.abs(act) + 1e-4 * K / 256), impl


def test_bounded_wait_gives_up_and_reports(B):
    """Every device-side wait of the library has a limit after which the kernel records the fact and
    returns.  The probe runs that wait on a barrier nothing signals, with a 1 ms limit instead of the
    library's second: the call reports ECHO_ERR_TIMEOUT, the warp waited about the limit, and the
    device is fine afterwards (nothing hung, nothing faulted)."""
    rc, waited = B.echo_debug_wait_limit(1_000_000)
    assert rc == -8
    assert 1_000_000 <= waited < 50_000_000
    rc, waited2 = B.echo_debug_wait_limit(200_000)
    assert rc == -8 and waited2 < waited + 5_000_000
    x = torch.arange(8, device="cuda")
    assert int(x.sum().item()) == 28                     # the context still answers


def test_group_advantage_matches_oracle(B):
    for P, G, seed in [(4, 4, 0), (32, 8, 1), (1, 2, 2), (7, 33, 3), (100, 16, 4)]:
        r = synth.make_rewards(P, G, seed)
        got = B.echo_group_advantage(torch.from_numpy(r).cuda()).cpu().numpy()
        want = o_adv.group_advantage(r)
        assert np.allclose(got, want, rtol=2e-5, atol=2e-5)
    r = np.full((3, 5), 0.25, dtype=np.float32)
    assert np.all(B.echo_group_advantage(torch.from_numpy(r).cuda()).cpu().numpy() == 0)
    with pytest.raises(B.EchoError):
        B.echo_group_advantage(torch.zeros((4, 1), device="cuda"))


def test_grpo_surrogate_matches_oracle(B):
    from oracle import objective
    rng = np.random.default_rng(17)
    for n, T, with_mask in [(1, 1, False), (5, 33, True), (64, 2048, True), (256, 100, False)]:
        ln, lo, ls = (-rng.exponential(1.0, size=(n, T)).astype(np.float32) for _ in range(3))
        adv = rng.normal(size=n).astype(np.float32)
        mask = (rng.random((n, T)) < 0.6).astype(np.uint8) if with_mask else None
        if with_mask and n > 2:
            mask[2] = 0
        got = B.echo_grpo_surrogate(*(torch.from_numpy(x).cuda() for x in (ln, lo, ls, adv)),
                                    torch.from_numpy(mask).cuda() if with_mask else None, 0.2, 1.7).cpu().numpy()
        want = objective.grpo_surrogate(ln, lo, ls, adv, mask if with_mask else np.ones((n, T)), 0.2, 1.7)
        assert np.allclose(got, want, rtol=2e-5, atol=2e-5)
        # with the KL regulariser against a reference policy
        lr = (ln + rng.normal(0, 0.3, size=(n, T))).astype(np.float32)
        got = B.echo_grpo_objective(*(torch.from_numpy(x).cuda() for x in (ln, lo, ls, lr, adv)),
                                    torch.from_numpy(mask).cuda() if with_mask else None, 0.2, 1.7, 0.04).cpu().numpy()
        want = objective.grpo_objective(ln, lo, ls, lr, adv, mask if with_mask else np.ones((n, T)), 0.2, 1.7, 0.04)
        assert np.allclose(got, want, rtol=2e-5, atol=2e-5)
