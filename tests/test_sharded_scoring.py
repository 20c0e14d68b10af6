"""Token-sharded and layer-streaming calibration on CPU: two gloo ranks on 127.0.0.1.  The control flow under
test is the product's (paper_2401_04044_b200/sharded.py); the numbers come from the oracle, so what is checked is
that shards, batches, the one all-reduce per layer and the finalisation reproduce the unsharded Eq. 3 scores, and
that every rank ends up with the same heavy-hitter set."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _layer(seed, d, m):
    rng = np.random.default_rng(seed)
    W1 = rng.standard_normal((d, m)) * 0.05
    W2 = rng.standard_normal((m, d)) * 0.05
    b1 = rng.standard_normal(m) * 0.1
    plant = rng.choice(m, 8, replace=False)
    W2[plant] *= 10
    b1[plant] += 1
    return W1, b1, W2, np.sort(plant)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import ffsplit_oracle as orc
    from paper_2401_04044_b200 import sharded
    d, m, T, k = 24, 96, 301, 8
    X = np.random.default_rng(5).standard_normal((T, d))          # the whole calibration set, the same on both ranks
    # ---- one layer, token-sharded: rank r scores tokens [lo, hi) in batches of 64
    W1, b1, W2, plant = _layer(1, d, m)
    energy = torch.zeros(m, dtype=torch.float64)
    scores = torch.zeros(m, dtype=torch.float64)
    calls = []

    def score_batch(a, b, acc):
        e, _, _ = orc.neuron_scores(X[a:b], W1, b1, W2, "gelu_erf")
        calls.append((a, b, acc))
        if acc:
            energy.add_(torch.from_numpy(e))
        else:
            energy.copy_(torch.from_numpy(e))

    def finalize():
        scores.copy_(energy * torch.from_numpy(np.sum(W2 * W2, axis=1)))

    n = sharded.score_token_sharded(score_batch, finalize, energy, T, 64)
    heavy, _ = orc.select_heavy(scores.numpy(), k)
    # ---- a stack of three layers, streaming: every rank pushes its share of each batch through the stack
    layers = [_layer(10 + l, d, m) for l in range(3)]
    energies = [torch.zeros(m, dtype=torch.float64) for _ in layers]
    stack_scores = [None] * 3
    lo, hi = sharded.shard_bounds(T, world, rank)
    my_batches = [X[a:b] for a, b in sharded.batches(lo, hi, 50)]

    def score_layer(l, x, acc):
        e, _, _ = orc.neuron_scores(x, layers[l][0], layers[l][1], layers[l][2], "gelu_erf")
        energies[l].copy_(energies[l] + torch.from_numpy(e) if acc else torch.from_numpy(e))

    def forward_layer(l, x):
        y = orc.dense_ffn(x, layers[l][0], layers[l][1], layers[l][2], None, "gelu_erf")
        return y[:, :d] if y.shape[1] >= d else y

    def finalize_layer(l):
        stack_scores[l] = (energies[l] * torch.from_numpy(np.sum(layers[l][2] ** 2, axis=1))).numpy().copy()

    seen = sharded.calibrate_stack_streaming(3, my_batches, score_layer, forward_layer, energies, finalize_layer)
    dist.barrier()
    out.put((rank, n, calls, scores.numpy().copy(), heavy, seen, stack_scores))
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_scores_and_agree_on_the_heavy_set():
    from oracle import ffsplit_oracle as orc
    from paper_2401_04044_b200 import sharded
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() + 7) % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((out.get(timeout=180) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    d, m, T, k = 24, 96, 301, 8
    X = np.random.default_rng(5).standard_normal((T, d))
    W1, b1, W2, plant = _layer(1, d, m)
    _, _, s_ref = orc.neuron_scores(X, W1, b1, W2, "gelu_erf")
    heavy_ref, _ = orc.select_heavy(s_ref, k)
    assert np.array_equal(heavy_ref, plant)
    assert got[0][1] + got[1][1] == T                              # the shards cover the set exactly once
    covered = sorted((a, b) for r in got for a, b, _ in r[2])
    assert covered[0][0] == 0 and covered[-1][1] == T and all(covered[i][1] == covered[i + 1][0] for i in range(len(covered) - 1))
    assert all(acc == (i > 0) for r in got for i, (_, _, acc) in enumerate(r[2]))   # first batch overwrites, the rest add
    for r in got:
        assert np.allclose(r[3], s_ref, rtol=1e-12, atol=0)
        assert np.array_equal(r[4], heavy_ref)
    assert np.array_equal(got[0][3], got[1][3])                    # bitwise the same scores on both ranks
    # the streamed stack: each layer's scores equal those of the whole set pushed through the dense layers
    layers = [_layer(10 + l, d, m) for l in range(3)]
    x = X
    for l in range(3):
        _, _, s_l = orc.neuron_scores(x, layers[l][0], layers[l][1], layers[l][2], "gelu_erf")
        for r in got:
            assert np.allclose(r[6][l], s_l, rtol=1e-10, atol=0)
        assert np.array_equal(got[0][6][l], got[1][6][l])
        x = orc.dense_ffn(x, layers[l][0], layers[l][1], layers[l][2], None, "gelu_erf")[:, :d]
    assert got[0][5] == len(sharded.batches(*sharded.shard_bounds(T, 2, 0), 50))


def test_shard_bounds_and_batches_cover_every_token_once():
    from paper_2401_04044_b200 import sharded
    for T in (0, 1, 7, 64, 65536 + 3):
        for world in (1, 2, 3, 8):
            spans = [sharded.shard_bounds(T, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == T
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            assert max(b - a for a, b in spans) - min(b - a for a, b in spans) <= 1
    assert sharded.batches(3, 10, 4) == [(3, 7), (7, 10)] and sharded.batches(5, 5, 4) == []


def test_single_process_flow_needs_no_process_group():
    from paper_2401_04044_b200 import sharded
    energy = torch.zeros(4)
    log = []
    n = sharded.score_token_sharded(lambda a, b, acc: (log.append((a, b, acc)), energy.add_(b - a))[1],
                                    lambda: log.append("fin"), energy, 10, 4)
    assert n == 10 and log == [(0, 4, False), (4, 8, True), (8, 10, True), "fin"] and energy.tolist() == [10.0] * 4
