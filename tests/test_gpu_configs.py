"""The large configurations, in the launch configuration the benchmark uses, checked where the CPU checker can still
follow (a chunk, a sub-batch) and otherwise through properties that hold at any size: the closed form for all-zero
weights, additivity over chunks of patterns (Section 4.3) and bitwise repeatability."""
import math

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, GpuNet, dev

pytestmark = pytest.mark.gpu


def _device_batch(seed, sizes, n, offset=0):
    X = torch.empty(n, sizes[0], device="cuda"); y = torch.empty(n, dtype=torch.int32, device="cuda")
    ul.fill_uniform(X, X.numel(), seed, si.TID_X, offset * sizes[0], 0)
    ul.fill_labels(y, n, seed, si.TID_LABELS, offset, sizes[-1])
    return X, y


def _rel(a, b):
    return oracle.rel_l2(a, b)


# ------------------------------------------------------------------ config 5: 1024-4096-4096-3203, 131072 patterns, seed 4
SIZES5 = [1024, 4096, 4096, 3203]
N5 = 131072


@pytest.mark.parametrize("math_mode", [ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16])
def test_config5_sub_batch_against_checker(math_mode):
    # the first 768 patterns of the seeded batch, through a handle sized for the full batch
    n = 768
    Ws, bs = si.mlp_params(4, SIZES5)
    X, y = si.mlp_batch(4, SIZES5, n)
    want = oracle.mlp_gradient(Ws, bs, X, y)
    g = GpuNet(SIZES5, math_mode, N5); g.set_params(Ws, bs)
    loss, dW, db = g.gradient(X, y)
    tol = TOL[math_mode]
    assert abs(loss - want[0]) <= tol * abs(want[0])
    for a, b in zip(dW + db, want[1] + want[2]):
        assert _rel(a, b) <= tol


def test_config5_full_batch_properties():
    g = GpuNet(SIZES5, ul.MATH_3XTF32, N5)
    X, y = _device_batch(4, SIZES5, N5)
    # (1) all-zero parameters: loss = n ln(n_o), db_L = n/n_o - counts, every other gradient zero
    g.set_params([np.zeros((SIZES5[l + 1], SIZES5[l]), np.float32) for l in range(3)],
                 [np.zeros(SIZES5[l + 1], np.float32) for l in range(3)])
    loss, dW, db = g.gradient(X, y)
    assert abs(loss - N5 * math.log(3203)) <= 1e-6 * loss
    assert all(np.all(w == 0) for w in dW) and np.all(db[0] == 0) and np.all(db[1] == 0)
    counts = np.bincount(y.cpu().numpy(), minlength=3203)
    assert np.allclose(db[2], N5 / 3203 - counts, atol=1e-3)
    # (2) seeded parameters: the whole batch equals four accumulated chunks (one of them ragged), and repeats bitwise
    Ws, bs = si.mlp_params(4, SIZES5)
    g.set_params(Ws, bs)
    whole = g.gradient(X, y)
    again = g.gradient(X, y)
    assert whole[0] == again[0] and all(np.array_equal(a, b) for a, b in zip(whole[1] + whole[2], again[1] + again[2]))
    cuts = [0, 40000, 80000, 100001, N5]
    for i in range(4):
        parts = g.gradient(X[cuts[i]:cuts[i + 1]], y[cuts[i]:cuts[i + 1]], accumulate=(i > 0))
    assert abs(parts[0] - whole[0]) <= 1e-6 * abs(whole[0])
    for a, b in zip(parts[1] + parts[2], whole[1] + whole[2]):
        assert _rel(a, b) <= 2e-5          # both sides carry the 1e-5 budget
    assert whole[0] > N5 * 0.9 * math.log(3203)


# ------------------------------------------------------------------ config 4: full epoch, 9,000,000 patterns, seed 3
SIZES4 = [400, 480, 3203]
N4 = 9_000_000
CHUNK4 = 131072


def test_config4_epoch_accumulation():
    Ws, bs = si.mlp_params(3, SIZES4)
    g = GpuNet(SIZES4, ul.MATH_3XTF32, CHUNK4); g.set_params(Ws, bs)
    X, y = _device_batch(3, SIZES4, N4)                      # 14.4 GB of patterns, resident
    starts = list(range(0, N4, CHUNK4))
    assert len(starts) == 69 and N4 - starts[-1] == 87104

    def epoch():
        for i, lo in enumerate(starts):
            hi = min(N4, lo + CHUNK4)
            g.net.gradient(g.W, g.b, X[lo:hi], SIZES4[0], y[lo:hi], hi - lo, i > 0, g.dW, g.db, g.loss)
        torch.cuda.synchronize()
        return float(g.loss.item()), [t.cpu().numpy() for t in g.dW + g.db]

    loss_a, grads_a = epoch()
    loss_b, grads_b = epoch()
    assert loss_a == loss_b and all(np.array_equal(a, b) for a, b in zip(grads_a, grads_b))      # bitwise repeatable

    # per-chunk gradients summed on the host in double, in chunk order, against the accumulator on the device
    tot = [np.zeros(t.shape, np.float64) for t in grads_a]; tot_loss = 0.0
    first = last = None
    for lo in starts:
        hi = min(N4, lo + CHUNK4)
        l, dW, db = g.gradient(X[lo:hi], y[lo:hi])
        tot_loss += l
        for t, c in zip(tot, dW + db):
            t += c
        if lo == 0: first = (l, dW, db)
        if hi == N4: last = (l, dW, db)
    assert abs(loss_a - tot_loss) <= 1e-9 * tot_loss
    for a, t in zip(grads_a, tot):
        assert _rel(a, t) <= 2e-6
    assert abs(loss_a / N4 - math.log(3203)) < 0.5

    # the checker on the first chunk and on the ragged last chunk (same seeded stream, generated on the host)
    for (l, dW, db), lo in ((first, 0), (last, starts[-1])):
        n = min(N4, lo + CHUNK4) - lo
        Xh, yh = si.mlp_batch(3, SIZES4, n, offset=lo)
        want = oracle.mlp_gradient(Ws, bs, Xh, yh)
        assert abs(l - want[0]) <= 1e-5 * abs(want[0])
        for a, b in zip(dW + db, want[1] + want[2]):
            assert _rel(a, b) <= 1e-5

    # then one plain step on the summed gradient, lr = 1e-3 (Section 4.2)
    loss_c, grads_c = epoch()
    g.net.sgd_step(g.W, g.b, g.dW, g.db, 1e-3)
    torch.cuda.synchronize()
    for w_new, w_old, gr in zip(g.W + g.b, Ws + bs, grads_c):
        want = oracle.sgd_step(w_old.ravel(), gr.ravel(), float(np.float32(1e-3)))
        got = w_new.cpu().numpy().ravel()
        assert np.all(np.abs(got - want) <= np.spacing(np.abs(want)))
