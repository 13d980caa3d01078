"""GPU parity: twn_sgd_update (Algorithm 1, UpdateParameters) and twn_ternarize_codes against the oracle.

Bar: updated weights and momentum bit-exact (the update is a fixed sequence of fp32 operations);
the threshold of the updated weights within 1e-12 relative; codes and counts bit-exact.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import twn
from _gpu_util import dev_f32, host_u32, workspace

pytestmark = pytest.mark.gpu

REL = 1e-12


@pytest.mark.parametrize("rows,cols", [(1, 1), (1, 3), (1, 1027), (64, 576), (10, 1024), (3, 5), (1, 300001), (512, 4608)])
def test_update_then_codes_match_the_oracle(rows, cols):
    n = rows * cols
    W = dg.he_normal(61, f"sgd{rows}x{cols}", rows, cols)
    g = dg.draw(61, f"sgdg{rows}x{cols}", n, "normal", 0.0, 0.05).reshape(rows, cols)
    V = dg.draw(61, f"sgdv{rows}x{cols}", n, "normal", 0.0, 0.05).reshape(rows, cols)
    Wd, gd, Vd = dev_f32(W), dev_f32(g), dev_f32(V)
    stats = twn.new_stats()
    ws = workspace(twn.ternarize_workspace_bytes())
    lr, mu, wd = 0.1, 0.9, 1e-4
    Wr, Vr = W, V
    for step in range(3):                       # several steps: the momentum buffer carries over
        twn.sgd_update(Wd, gd, Vd, lr, mu, wd, 0.7, stats, ws)
        Wr, Vr = oracle.sgd_update(Wr, g, Vr, lr, mu, wd)
    torch.cuda.synchronize()
    assert np.array_equal(Wd.cpu().numpy().view(np.uint32), Wr.view(np.uint32))
    assert np.array_equal(Vd.cpu().numpy().view(np.uint32), Vr.view(np.uint32))
    ref, ref_codes = oracle.ternarize(Wr, 0.7)
    st = twn.stats_to_host(stats)
    assert st["status"] == 0 and ref.n_boundary == 0
    assert abs(st["delta"] - ref.delta) <= REL * ref.delta
    assert abs(st["sum_abs"] - ref.sum_abs) <= REL * ref.sum_abs
    # the coding sweep alone, against that threshold
    ld = twn.ld_for(cols)
    packed = torch.full((rows, ld // 16), -1, dtype=torch.int32, device="cuda")
    codes = torch.full((rows, cols), 7, dtype=torch.int8, device="cuda")
    twn.ternarize_codes(Wd, rows, cols, stats, packed, ld, codes, ws)
    st = twn.stats_to_host(stats)
    assert abs(st["alpha"] - ref.alpha) <= REL * ref.alpha and abs(st["delta"] - ref.delta) <= REL * ref.delta
    assert (st["n_neg"], st["n_zero"], st["n_pos"]) == (ref.n_neg, ref.n_zero, ref.n_pos)
    assert np.array_equal(host_u32(packed), oracle.pack(ref_codes.reshape(rows, cols), ld))
    assert np.array_equal(codes.cpu().numpy(), ref_codes.reshape(rows, cols))
    # and the same codes as a full ternarization of the updated weights
    stats2 = twn.new_stats()
    packed2 = torch.empty_like(packed)
    twn.ternarize(Wd, 0.7, stats2, packed2, ld, None, ws, rows=rows, cols=cols)
    assert torch.equal(packed, packed2)


def test_update_without_stats_and_with_plain_descent():
    W = dg.he_normal(62, "sgd-plain", 1, 4096).reshape(-1)
    g = dg.draw(62, "sgd-plain-g", 4096, "normal", 0.0, 0.05)
    Wd, gd, Vd = dev_f32(W), dev_f32(g), dev_f32(np.zeros(4096, np.float32))
    ws = workspace(twn.ternarize_workspace_bytes())
    twn.sgd_update(Wd, gd, Vd, 0.5, 0.0, 0.0, 0.7, None, ws)
    Wr, Vr = oracle.sgd_update(W, g, np.zeros(4096, np.float32), 0.5, 0.0, 0.0)
    assert np.array_equal(Wd.cpu().numpy(), Wr) and np.array_equal(Vd.cpu().numpy(), g)


def test_nonfinite_update_is_flagged_and_arguments_are_checked():
    W = np.ones(64, np.float32)
    g = np.zeros(64, np.float32); g[7] = np.inf
    Wd, gd, Vd = dev_f32(W), dev_f32(g), dev_f32(np.zeros(64, np.float32))
    stats = twn.new_stats()
    ws = workspace(twn.ternarize_workspace_bytes())
    twn.sgd_update(Wd, gd, Vd, 0.1, 0.9, 0.0, 0.7, stats, ws)
    assert twn.stats_to_host(stats)["status"] == -4
    with pytest.raises(twn.TwnError):
        twn.sgd_update(Wd, gd, Vd, float("nan"), 0.9, 0.0, 0.7, stats, ws)
    with pytest.raises(twn.TwnError):
        twn.sgd_update(Wd, gd, Vd, 0.1, 0.9, 0.0, 0.7, stats, torch.empty(256, dtype=torch.uint8, device="cuda"))
