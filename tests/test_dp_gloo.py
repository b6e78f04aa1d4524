"""Training-set parallelism (Section 4.3) on two CPU ranks over gloo: each rank evaluates its slice of the seeded
pattern stream with the CPU checker, the gradients are summed through the package's exchange, and every rank must
end up with the gradient of the whole batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import dp

SIZES = [12, 9, 5]
PER_RANK = 37
SEED = 31


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir, ordered=False):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Ws, bs = si.mlp_params(SEED, SIZES)
        first, last = dp.shard_range(rank, world, PER_RANK)
        X, y = si.mlp_batch(SEED, SIZES, last - first, offset=first)
        loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
        grads = [torch.from_numpy(np.ascontiguousarray(g)) for g in dW + db]       # float64 on the CPU
        loss_t = torch.tensor([loss], dtype=torch.float64)
        ex = dp.GradientExchange(grads, dist, ordered=ordered)
        ex.all_reduce(grads, loss_t)
        np.savez(os.path.join(out_dir, "rank%d.npz" % rank), loss=loss_t.numpy(), *[g.numpy() for g in grads])
    finally:
        dist.destroy_process_group()


def test_two_ranks_sum_to_the_full_batch(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    Ws, bs = si.mlp_params(SEED, SIZES)
    X, y = si.mlp_batch(SEED, SIZES, world * PER_RANK)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    for rank in range(world):
        got = np.load(os.path.join(str(tmp_path), "rank%d.npz" % rank))
        assert abs(got["loss"][0] - loss) <= 1e-12 * abs(loss)
        for i, ref in enumerate(dW + db):
            assert np.allclose(got["arr_%d" % i], ref, rtol=1e-12, atol=1e-14)


def test_ordered_exchange_is_the_rank_order_sum_on_every_rank(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path), True), nprocs=world, join=True)
    Ws, bs = si.mlp_params(SEED, SIZES)
    per_rank = []
    for rank in range(world):
        first, last = dp.shard_range(rank, world, PER_RANK)
        X, y = si.mlp_batch(SEED, SIZES, last - first, offset=first)
        per_rank.append(oracle.mlp_gradient(Ws, bs, X, y))
    got = [np.load(os.path.join(str(tmp_path), "rank%d.npz" % rank)) for rank in range(world)]
    assert got[0]["loss"][0] == got[1]["loss"][0] == per_rank[0][0] + per_rank[1][0]
    n_tensors = 2 * (len(SIZES) - 1)
    for i in range(n_tensors):
        a0 = (per_rank[0][1] + per_rank[0][2])[i]; a1 = (per_rank[1][1] + per_rank[1][2])[i]
        assert np.array_equal(got[0]["arr_%d" % i], got[1]["arr_%d" % i])       # bitwise the same on both ranks
        assert np.array_equal(got[0]["arr_%d" % i], a0 + a1)                     # and exactly rank 0's plus rank 1's


def test_shard_arithmetic():
    assert dp.shard_range(0, 4, 10) == (0, 10) and dp.shard_range(3, 4, 10) == (30, 40)
    cover = [dp.split_range(163480, 8, r) for r in range(8)]             # a pattern count of Section 6.3
    assert cover[0][0] == 0 and cover[-1][1] == 163480
    assert all(a[1] == b[0] for a, b in zip(cover, cover[1:]))
    assert max(b - a for a, b in cover) - min(b - a for a, b in cover) <= 1
    with pytest.raises(ValueError):
        dp.shard_range(4, 4, 10)


def test_single_rank_exchange_is_a_no_op():
    g = [torch.arange(6, dtype=torch.float32).reshape(2, 3), torch.ones(4)]
    before = [t.clone() for t in g]
    loss = torch.tensor([2.5], dtype=torch.float64)
    dp.GradientExchange(g, None).all_reduce(g, loss)
    assert all(torch.equal(a, b) for a, b in zip(g, before)) and loss.item() == 2.5


# ---- fixed total number of patterns (the processor-scaling experiment of Section 6.3) and the exchange launched
# ---- layer by layer while the rest of the gradient is still being computed (Section 5.2)

TOTAL = 75          # not a multiple of the world size: the first rank gets one pattern more


def _worker_strong(rank, world, port, out_dir, ordered, overlapped):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Ws, bs = si.mlp_params(SEED, SIZES)
        first, last = dp.split_range(TOTAL, world, rank)
        X, y = si.mlp_batch(SEED, SIZES, last - first, offset=first)
        loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
        grads = [torch.from_numpy(np.ascontiguousarray(g)) for g in dW + db]
        loss_t = torch.tensor([loss], dtype=torch.float64)
        L = len(SIZES) - 1
        if overlapped:
            ex = dp.GradientExchange(grads, dist, ordered=ordered, groups=dp.layer_groups(L))
            for g in range(L - 1):           # the top layers' gradients leave early, the last group leaves in finish()
                ex.start(g, grads)
            ex.finish(grads, loss_t)
        else:
            ex = dp.GradientExchange(grads, dist, ordered=ordered)
            ex.all_reduce(grads, loss_t)
        np.savez(os.path.join(out_dir, "rank%d_%d.npz" % (rank, int(overlapped))), loss=loss_t.numpy(), first=first, last=last,
                 *[g.numpy() for g in grads])
    finally:
        dist.destroy_process_group()


def test_layer_groups_follow_the_order_in_which_gradients_become_final():
    assert dp.layer_groups(2) == [[1, 3], [0, 2]]
    assert dp.layer_groups(3) == [[2, 5], [1, 4], [0, 3]]
    with pytest.raises(ValueError):
        dp.GradientExchange([torch.zeros(2), torch.zeros(3)], None, groups=[[0]])


@pytest.mark.parametrize("ordered", [False, True])
def test_fixed_total_split_and_overlapped_exchange_give_the_serial_bits(tmp_path, ordered):
    world = 2
    for overlapped in (False, True):
        mp.spawn(_worker_strong, args=(world, _free_port(), str(tmp_path), ordered, overlapped), nprocs=world, join=True)
    Ws, bs = si.mlp_params(SEED, SIZES)
    X, y = si.mlp_batch(SEED, SIZES, TOTAL)
    loss, dW, db = oracle.mlp_gradient(Ws, bs, X, y)
    serial = [np.load(os.path.join(str(tmp_path), "rank%d_0.npz" % r)) for r in range(world)]
    over = [np.load(os.path.join(str(tmp_path), "rank%d_1.npz" % r)) for r in range(world)]
    assert [(int(s["first"]), int(s["last"])) for s in serial] == [(0, 38), (38, 75)]       # uneven remainder
    for r in range(world):
        assert abs(serial[r]["loss"][0] - loss) <= 1e-12 * abs(loss)
        assert over[r]["loss"][0] == serial[r]["loss"][0]
        for i, ref in enumerate(dW + db):
            assert np.allclose(serial[r]["arr_%d" % i], ref, rtol=1e-12, atol=1e-14)
            # launched group by group or in one go: the same additions, the same bits
            assert np.array_equal(over[r]["arr_%d" % i], serial[r]["arr_%d" % i])
            if ordered:
                assert np.array_equal(over[0]["arr_%d" % i], over[1]["arr_%d" % i])
