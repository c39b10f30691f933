"""Encoder block around the mixed GEMMs: the quantized linears with fp16 in and out, calibrated on the
block's own activations; stock fp16 operators between them (not part of the method's hot path)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_02822_b200 import binding as fx
from paper_2510_02822_b200 import vit_block

pytestmark = pytest.mark.gpu


def test_block_runs_and_its_linears_match_the_oracle():
    dev = torch.device("cuda:0")
    blk = vit_block.Block("deits", 2, dev)
    outs = {}
    for ratio in (0.0, 1.0, 0.0):
        blk.set_ratio(ratio)
        y = blk.forward()
        torch.cuda.synchronize()
        assert bool(torch.isfinite(y).all())
        outs.setdefault(ratio, []).append(y.clone())
    assert torch.equal(outs[0.0][0], outs[0.0][1])          # same ratio, same bits
    assert not torch.equal(outs[0.0][0], outs[1.0][0])      # 4-bit groups change the result
    # the first linear (QKV) on the block's own fp16 activations, against the oracle, fp16 output bit for bit
    blk.set_ratio(0.5)
    h = torch.nn.functional.layer_norm(blk.x, (blk.D,), blk.ln[0], blk.ln[1])
    got = blk.linear("qkv", h).cpu().numpy()
    L, x_scale, _slab, _Y, Wq = blk.layers["qkv"]
    Wq_h = Wq.cpu().numpy()
    q = oracle.quantize(h.float().cpu().numpy(), x_scale)
    # the handle's order and positions come from the device calibration: recompute them with the oracle
    lo, hi = oracle.channel_ranges(q)
    sx_group = oracle.static_positions(lo, hi, 16)
    perm, _ = oracle.greedy_order(lo, hi, oracle.weight_absmax_linear(Wq_h), 16)
    sw = oracle.weight_positions_linear(Wq_h, 16, perm)
    acc = oracle.mixed_gemm_acc(q, Wq_h, 16, perm, sx_group[perm].copy(), sw, oracle.n_low(0.5, blk.D // 16))
    from paper_2510_02822_b200 import inputs
    c = inputs.vit_linear("blk_qkv", 256, blk.D, 3 * blk.D, 16, seed=11000)
    want = oracle.epilogue_f16(acc, x_scale, c.w_scale, c.bias)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    fx.flexiq_check_status()
    blk.close()
