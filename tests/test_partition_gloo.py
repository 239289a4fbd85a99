"""Multi-rank host logic on CPU (gloo, world_size 2): candidate sharding, local regeneration of a rank's
candidates from <seed, k>, and the <seed, reward> exchange of Algorithm 1 line 11."""
import os
import socket

import numpy as np
import pytest

from paper_2507_04453_b200 import partition, workloads as wl


def test_partition_covers_and_balances():
    rng = np.random.default_rng(0)
    for P, W in [(64, 2), (64, 8), (5, 8), (1, 2), (256, 4)]:
        lens = rng.integers(0, 1025, size=P)
        off = np.concatenate([[0], np.cumsum(lens)])
        parts = partition.partition_candidates(off, W)
        assert len(parts) == W and parts[0][0] == 0 and parts[-1][1] == P
        assert all(parts[g][1] == parts[g + 1][0] for g in range(W - 1))
        tok = [int(off[b] - off[a]) for a, b in parts]
        assert sum(tok) == int(off[-1])
        if P >= 8 * W:
            assert max(tok) - min(tok) <= 2 * 1024  # within two longest segments of each other
    assert partition.partition_candidates([0, 0, 0, 0], 2) == [(0, 1), (1, 3)]
    assert list(partition.local_offsets([0, 4, 6, 9], 1, 3)) == [0, 2, 5]
    msg = partition.pack_seed_reward(0x1_0000_0007, 0.5)
    assert msg.nbytes == 8 and msg[0] == 7 and msg[1:].view(np.float32)[0] == 0.5


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    import torch
    from oracle import essa_oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = wl.scaled_config("4", d_model=64, d_kv=64, rank=4, P=10, seg_len=9)
        off = wl.make_segments(cfg)
        adapters = [wl.make_adapter(cfg, i) for i in range(4)]
        cma = wl.make_cma_state(cfg, adapters)
        k0, k1 = partition.partition_candidates(off, world)[rank]
        # each rank regenerates only its own members (what essa_sample_population_range does on a GPU)
        mine = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, k1 - k0, k_begin=k0)
        # each rank projects its own tokens; rewards stand in for F(x)
        ad = adapters[0]
        x = wl.make_tokens(cfg, 0, int(off[-1]))[off[k0]:off[k1]]
        y = orc.apply_projection(ad.W0, ad.U_A, ad.V_A, ad.U_B, ad.V_B, x, partition.local_offsets(off, k0, k1),
                                 mine, 0, 4, 4)
        rewards = np.array([y[a:b].sum() for a, b in zip(partition.local_offsets(off, k0, k1)[:-1],
                                                        partition.local_offsets(off, k0, k1)[1:])], dtype=np.float32)
        # exchange <seed, reward>: 8 bytes per candidate, padded to the largest shard
        maxc = max(b - a for a, b in partition.partition_candidates(off, world))
        msg = np.zeros((maxc, 2), dtype=np.int32)
        for j in range(k1 - k0):
            msg[j] = partition.pack_seed_reward(cma.seed + k0 + j, float(rewards[j])).view(np.int32)
        gathered = [torch.zeros((maxc, 2), dtype=torch.int32) for _ in range(world)]
        dist.all_gather(gathered, torch.from_numpy(msg))
        q.put((rank, k0, k1, mine, y, [g.numpy() for g in gathered]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_regenerate_and_exchange():
    import torch.multiprocessing as mp
    from oracle import essa_oracle as orc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=120) for _ in procs], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = wl.scaled_config("4", d_model=64, d_kv=64, rank=4, P=10, seg_len=9)
    off = wl.make_segments(cfg)
    adapters = [wl.make_adapter(cfg, i) for i in range(4)]
    cma = wl.make_cma_state(cfg, adapters)
    full = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    ad = adapters[0]
    y_full = orc.apply_projection(ad.W0, ad.U_A, ad.V_A, ad.U_B, ad.V_B, wl.make_tokens(cfg, 0, int(off[-1])), off,
                                  full, 0, 4, 4)
    assert res[0][1] == 0 and res[0][2] == res[1][1] and res[1][2] == cfg.P
    for rank, k0, k1, mine, y, gathered in res:
        assert np.array_equal(mine, full[k0:k1])            # same members, regenerated locally
        np.testing.assert_allclose(y, y_full[off[k0]:off[k1]], rtol=0, atol=1e-12)
        # every rank ends with the same <seed, reward> list, 8 bytes per candidate
        seeds = np.concatenate([g[:b - a, 0] for g, (_, a, b, *_r) in zip(gathered, res)])
        assert list(seeds) == [cma.seed + k for k in range(cfg.P)]
    assert all(np.array_equal(a, b) for a, b in zip(res[0][5], res[1][5]))
