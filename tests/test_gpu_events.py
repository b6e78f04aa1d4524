"""ulsnn_mlp_set_gradient_events: the per-layer "gradient is final" events that let the exchange between several GPUs
start on the top layer's gradient while the layers below are still being computed (Sections 4.3, 5.2).  On one GPU:
a second stream that waits for a layer's event and copies that layer's gradient must see the final values, the top
layer's event must come no later than the first layer's, and the results do not change."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from paper_1911_05181_b200 import binding as ul
from helpers import TOL, GpuNet, dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("math", [ul.MATH_3XTF32, ul.MATH_TF32, ul.MATH_BF16, ul.MATH_FP32_SIMT])
def test_layer_events_mark_final_gradients(math):
    sizes, n = [40, 64, 48, 33], 3000
    Ws, bs = si.mlp_params(9, sizes)
    X, y = si.mlp_batch(9, sizes, n)
    want = oracle.mlp_gradient(Ws, bs, X, y)
    g = GpuNet(sizes, math, n); g.set_params(Ws, bs)
    plain = g.gradient(X, y)                                     # without events
    L = len(sizes) - 1
    main = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    events = [torch.cuda.Event(enable_timing=True) for _ in range(L)]
    for e in events:
        e.record(main)                                           # an event exists once it has been recorded
    g.net.set_gradient_events(events)
    dX, dy = dev(X), dev(y)
    for t in g.dW + g.db:
        t.fill_(float("nan"))
    g.net.gradient(g.W, g.b, dX, sizes[0], dy, n, False, g.dW, g.db, g.loss)
    copies = [None] * (2 * L)
    with torch.cuda.stream(side):
        for w in range(L - 1, -1, -1):                           # the order in which the library finishes them
            side.wait_event(events[w])
            copies[w] = g.dW[w].clone(); copies[L + w] = g.db[w].clone()
    torch.cuda.synchronize()
    for w in range(L - 1):
        assert events[w + 1].elapsed_time(events[w]) >= 0.0      # a layer above is final no later than the one below
    got = [t.cpu().numpy() for t in copies]
    for a, b_, ref in zip(got, plain[1] + plain[2], want[1] + want[2]):
        assert np.array_equal(a, b_)                             # the copy taken at the event is the final gradient
        assert oracle.rel_l2(a, ref) <= TOL[math]
    g.net.set_gradient_events(None)
    again = g.gradient(X, y)
    assert all(np.array_equal(u, v) for u, v in zip(again[1] + again[2], plain[1] + plain[2]))
    g.net.close()
