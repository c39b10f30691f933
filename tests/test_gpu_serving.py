"""Serving loop on the GPU (Sec. 8): one CUDA graph per ratio replayed in any order after
flexiq_layer_sync_ratio, and the live queue around a small stack."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import inputs, serving
from tests import helpers

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    return torch.device("cuda:0")


def test_graphs_of_several_ratios_replay_in_any_order(dev):
    """A graph captured at ratio r stays valid after other ratios ran (the run-time ratio switch): with the ratio set
    again and flexiq_layer_sync_ratio called before the replay, as a deployment may do, and -- second loop -- with
    nothing at all between the replays."""
    case = inputs.ranged_linear("srv", 333, 512, 304, 16, seed=77, group_structured=True)
    perm, sxg, sxs, sw = helpers.prepare_linear(case)
    L = fx.Layer(torch.from_numpy(case.Wq).to(dev), torch.from_numpy(case.w_scale).to(dev), torch.from_numpy(case.bias).to(dev), perm, sxg, case.G)
    X = torch.from_numpy(case.X).to(dev)
    x4, x8 = L.alloc_slabs(case.M)
    Y = torch.empty((case.M, case.N), dtype=torch.int8, device=dev)
    q = oracle.quantize(case.X, case.x_scale)
    ratios = [0.0, 0.25, 0.5, 0.75, 1.0]
    want, graphs = {}, {}
    side = torch.cuda.Stream()

    def launch():
        fx.flexiq_quantize_lower(L.h, X, fx.DTYPE_F32, case.M, case.x_scale, 0, x4, x8)
        fx.flexiq_mixed_gemm(L.h, x4, x8, None, case.M, case.x_scale, case.y_scale, fx.OUT_REQUANT_I8, Y)

    for r in ratios:
        nl = oracle.n_low(r, case.K // case.G)
        acc = oracle.mixed_gemm_acc(q, case.Wq, case.G, perm, sxs, sw, nl)
        want[r] = oracle.epilogue_i8(acc, case.x_scale, case.w_scale, case.bias, case.y_scale)
        L.set_lowbit_ratio(r)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            launch()
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                launch()
        torch.cuda.synchronize()
        graphs[r] = g
    assert not np.array_equal(want[0.0], want[1.0])
    for r in [0.5, 0.0, 1.0, 0.25, 1.0, 0.75, 0.0]:
        L.set_lowbit_ratio(r)
        L.sync_ratio()
        Y.zero_()
        graphs[r].replay()
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy(), want[r]), r
    L.sync_ratio()  # nothing to write: a no-op
    for r in [0.75, 0.25, 1.0, 0.5, 0.25, 0.0]:   # nothing between the replays: every graph is complete in itself
        Y.zero_()
        graphs[r].replay()
        torch.cuda.synchronize()
        assert np.array_equal(Y.cpu().numpy(), want[r]), r
    fx.flexiq_check_status()
    L.close()


def test_live_queue_on_a_small_stack(dev):
    """Every batch of the trace runs on the GPU at the controller's level; the responses obey the
    queue's invariants and the stack still computes the oracle's values afterwards."""
    stack = serving.Stack("deits", 2, dev)
    table = serving.profile_service(stack, 2, 3)
    assert table.shape == (serving.LEVELS, 2) and np.all(table > 0)
    rates = np.array([100.0, 1000.0, 3000.0])
    lat = np.array([[table[l, 0] * (1.0 + r / 1000.0) for r in rates] for l in range(serving.LEVELS)])
    ctrl = fx.Controller(rates, lat, 1.5 * float(table[0, 0]), 0.02)
    arr = inputs.fluctuating_arrivals(5, 500.0, 1500.0, 0.2, 0.4)
    resp, lvl = serving.live(stack, ctrl, arr, 2, 0.02)
    done = arr + resp
    assert resp.size == arr.size and np.all(resp > 0)
    assert np.all(np.diff(done) >= -1e-12)
    assert lvl.min() >= 0 and lvl.max() < serving.LEVELS and len(set(lvl.tolist())) >= 2
    assert np.all(np.abs(np.diff(lvl)) <= 1)
    ctrl.close()
    # the first layer at the level the run ended on, against the oracle
    L, c, X, slab, Y = stack.inst[0]
    stack.run(2)
    torch.cuda.synchronize()
    perm, sxg, sxs, sw = helpers.prepare_linear(c)
    nl = oracle.n_low(stack.level / (serving.LEVELS - 1), c.K // c.G)
    q = oracle.quantize(c.X[:2 * 197], c.x_scale)
    acc = oracle.mixed_gemm_acc(q, c.Wq, c.G, perm, sxs, sw, nl)
    assert np.array_equal(Y[:2 * 197].cpu().numpy(), oracle.epilogue_i8(acc, c.x_scale, c.w_scale, c.bias, c.y_scale))
    fx.flexiq_check_status()
