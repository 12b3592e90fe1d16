"""The N > 1 path of the benchmark is N independent replicas: the job's prompt set is cut by prompt
(groups are never split), each rank numbers its sequences from its first prompt's global index, there
is no data-path collective, and the job's time is the slowest rank's.  Covered here with two gloo
ranks on the CPU (no GPU needed): the cut, drawn through the oracle's sampler with global sequence
ids, reproduces what one process draws for the whole set."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from oracle import advantage, sampler
    from paper_2602_02192_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # 7 prompts over 2 ranks: [0, 4) and [4, 7).  Every rank draws the first token of its own sequences
    # from the logits row of their prompt, with the GLOBAL sequence id p * G + g in the noise stream
    # (what echo_set_sequence_base(lo * G) makes the library do); gathered, the draws equal the ones a
    # single process makes for the whole set.
    n_prompts, G, V, seed = 7, 3, 257, 99
    logits = np.random.default_rng(5).normal(size=(n_prompts, V))
    lo, hi = bench.rank_prompt_range(n_prompts, rank, world)
    mine = torch.full((n_prompts * G,), -1, dtype=torch.int64)
    base = lo * G
    for p_local in range(hi - lo):
        for g in range(G):
            s_local = p_local * G + g
            mine[base + s_local] = sampler.draw(logits[lo + p_local], 1.0, seed, base + s_local, 0).token
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    stacked = torch.stack(gathered)
    covered_once = bool(((stacked >= 0).sum(dim=0) == 1).all())             # every sequence on exactly one rank
    whole = torch.tensor([sampler.draw(logits[s // G], 1.0, seed, s, 0).token for s in range(n_prompts * G)])
    distinct = covered_once and bool((stacked.max(dim=0).values == whole).all())
    # each rank is slower or faster; the job's time is the maximum
    elapsed = bench.max_over_ranks(100.0 * (rank + 1), "cpu", world)
    value = bench.job_tokens_per_second(4 * 4 * 32, world, 3, elapsed)
    # groups never cross ranks, so group-normalised rewards need nothing from another rank
    rewards = synth.make_rewards(4, 4, 7 + rank)
    adv_local = advantage.group_advantage(rewards)
    all_rewards = [torch.zeros(4, 4, dtype=torch.float32) for _ in range(world)]
    dist.all_gather(all_rewards, torch.from_numpy(rewards))
    adv_global = advantage.group_advantage(torch.cat(all_rewards).numpy())
    same_adv = np.allclose(adv_global[4 * rank: 4 * rank + 4], adv_local)
    dist.barrier()
    out[rank] = (distinct, elapsed, value, same_adv)
    dist.destroy_process_group()


def test_two_replica_ranks_on_gloo():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert len(out) == world
    for rank in range(world):
        distinct, elapsed, value, same_adv = out[rank]
        assert distinct and same_adv
        assert elapsed == 200.0                                   # max over ranks
        assert abs(value - 2 * 3 * 512 / 0.2) < 1e-6              # whole-job tokens / slowest rank's time


def test_reference_arm_is_rank_zero_only(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    bench.run_reference(type("A", (), {"workload": "tiny", "warmup": 1, "steps": 1, "gpus": 2})())
    assert capsys.readouterr().out == ""


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` on the tiny workload: one JSON line with the benchmark's keys."""
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


def _chain_worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2602_02192_b200 import chain, synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    shape = synth.SHAPES["tiny"]
    # rank 0 holds the new snapshot; ranks 1..3 are rollout replicas ranked by a peer score
    scores = [40.0, 90.0, 70.0]                                   # workers 0, 1, 2 = ranks 1, 2, 3
    chains = [[w + 1 for w in c] for c in chain.plan_chains(scores, 200.0, 100.0)]     # floor(200 / 100) = 2 chains
    flat = chain.pack(synth.make_weights(shape, 5), shape) if rank == 0 else None
    got, version = chain.disseminate(flat, 17, shape, 0, chains, chunk_bytes=64 << 10)
    want = chain.pack(synth.make_weights(shape, 5), shape)        # seeded: every rank can rebuild the bits
    same = bool(torch.equal(got, want))
    w = chain.unpack(got, shape)
    ref = synth.make_weights(shape, 5)
    views_ok = all(torch.equal(w[n][l], ref[n][l]) for n in chain.LAYER_TENSORS for l in range(shape.n_layers)) and \
        all(torch.equal(w[n], ref[n]) for n in chain.GLOBAL_TENSORS)
    aligned = all(w[n][l].data_ptr() % 16 == 0 for n in chain.LAYER_TENSORS for l in range(shape.n_layers))
    dist.barrier()
    out[rank] = (chains, version, same, views_ok, aligned)
    dist.destroy_process_group()


def test_snapshot_chain_dissemination_on_gloo():
    """Section 4.3 on four CPU ranks: the source streams the snapshot in 64 KiB chunks to the two seeds,
    the better seed's chain has a second hop that receives every chunk from the seed, not from the
    source; every replica ends with the snapshot bit for bit and the new version tag."""
    world = 4
    port = 31500 + os.getpid() % 2000
    mgr = mp.get_context("spawn").Manager()
    out = mgr.dict()
    mp.spawn(_chain_worker, args=(world, port, out), nprocs=world, join=True)
    assert len(out) == world
    for rank in range(world):
        chains, version, same, views_ok, aligned = out[rank]
        assert chains == [[2, 1], [3]]            # seeds: ranks 2 (score 90) and 3 (70); rank 1 behind the best seed
        assert version == 17 and same and views_ok and aligned


def test_chain_repair_closes_over_a_failed_relay():
    sys.path.insert(0, ROOT)
    from paper_2602_02192_b200 import chain
    chains = [[4, 1, 7, 2], [5, 3], [6]]
    assert chain.excise(chains, 1) == [[4, 7, 2], [5, 3], [6]]      # the tail reattaches to the nearest healthy parent
    assert chain.excise(chains, 4) == [[1, 7, 2], [5, 3], [6]]      # a failed seed: its child becomes the seed
    assert chain.excise(chains, 6) == [[4, 1, 7, 2], [5, 3]]        # a chain of one disappears
    assert chain.excise(chains, 9) == chains
