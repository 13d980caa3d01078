"""GPU parity of the chained workloads (LeNet-5, VGG-7, ResNet-18 shapes), layer by layer with
teacher forcing: the oracle's layer is fed the very bytes the GPU's layer consumed, and is
evaluated on sampled output pixels / gradient entries (all of them for small tensors).

bf16 outputs: |got - ref| <= tol + 2^-8 (|ref| + tol), tol = 1e-4 * alpha * |scale| * A + 1e-6
(the stated fp32 bound plus one bf16 rounding).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_1605_04711_b200 import datagen as dg
from paper_1605_04711_b200 import nets, twn

pytestmark = pytest.mark.gpu


def bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f64(t):
    if t.dtype == torch.bfloat16:
        return dg.bf16_bits_to_f64(bits(t))
    return t.cpu().numpy().astype(np.float64)


def sample(n, count, seed):
    if n <= count:
        return np.arange(n)
    rng = np.random.default_rng(seed)
    edge = np.concatenate([np.arange(64), np.arange(n - 64, n)])
    return np.unique(np.concatenate([edge, rng.integers(0, n, count)]))


def within(got, ref, tol, bf16):
    lim = tol + (2.0 ** -8) * (np.abs(ref) + tol) if bf16 else tol
    err = np.abs(got - ref)
    assert np.all(err <= lim), f"worst err/lim {np.max(err / lim):.3g}"


def layer_codes(net, L):
    W = L.extra["W"].cpu().numpy()
    st, codes = oracle.ternarize(W, net.delta_factor)
    got = twn.stats_to_host(L.extra["stats"])
    assert got["status"] == 0
    assert abs(got["alpha"] - st.alpha) <= 1e-12 * st.alpha and abs(got["delta"] - st.delta) <= 1e-12 * st.delta
    ld = L.extra["ld"]
    assert np.array_equal(L.extra["packed"].cpu().numpy().view(np.uint32), oracle.pack(codes.reshape(L.Cout, L.K), ld))
    return st.alpha, codes.reshape(L.Cout, L.k, L.k, L.Cin)


def check_forward(net, npix=160):
    for L in net.layers.values():
        alpha, codes = layer_codes(net, L)
        e = L.extra
        x = bits(net.act[L.src]).reshape(L.B, L.H, L.W, L.Cin)
        y = net.act[L.name]
        od = oracle.conv_desc(L.B, L.H, L.W, L.Cin, L.Cout, L.k, L.stride, L.pad)
        pix = sample(L.B * L.Ho * L.Wo, npix, 1)
        scale = e["scale"].cpu().numpy() if e["scale"] is not None else None
        shift = e["shift"].cpu().numpy() if e["shift"] is not None else None
        res = f64(net.act[L.residual]) if L.residual else None
        ref, A = oracle.conv2d_fwd(od, x, codes, alpha, scale, shift, res, L.relu, pixels=pix)
        tol = 1e-4 * alpha * A * (np.abs(scale.astype(np.float64)) if scale is not None else 1.0) + 1e-6
        got = f64(y).reshape(-1, L.Cout)[pix]
        within(got, ref, tol, y.dtype == torch.bfloat16)


def check_pools(net, images=2):
    for op in net.ops:
        if op[0] == "maxpool":
            _, name, src, k, s, p = op
            x = f64(net.act[src][:images])
            yr, _ = oracle.maxpool(x, k, s, p)
            assert np.array_equal(f64(net.act[name][:images]), yr)
        elif op[0] == "avgpool":
            _, name, src = op
            yr = oracle.global_avgpool(f64(net.act[src]))
            got = f64(net.act[name]).reshape(yr.shape)
            assert np.all(np.abs(got - yr) <= 2.0 ** -8 * np.abs(yr) + 1e-6)


def check_backward(net, npix=96, nent=200):
    for L in net.layers.values():
        alpha, codes = layer_codes(net, L)
        e = L.extra
        od = oracle.conv_desc(L.B, L.H, L.W, L.Cin, L.Cout, L.k, L.stride, L.pad)
        dz = bits(e["dz"]).reshape(L.B, L.Ho, L.Wo, L.Cout)
        x = bits(net.act[L.src]).reshape(L.B, L.H, L.W, L.Cin)
        # straight-through weight gradient
        ent = sample(L.Cout * L.K, nent, 2)
        ref, A = oracle.conv2d_bwd_weight(od, x, dz, entries=ent)
        dW = e["dW"].cpu().numpy().astype(np.float64)
        got = dW[:, :L.K].reshape(-1)[ent]
        within(got, ref, 1e-4 * A + 1e-6, False)
        # backward for data, including the contribution that was already in the buffer
        if L.src == "input":
            continue
        pix = sample(L.B * L.H * L.W, npix, 3)
        ref, A = oracle.conv2d_bwd_data(od, dz, codes, alpha, pixels=pix)
        tol = 1e-4 * alpha * A + 1e-6
        got = f64(net.grad_of_input[L.name]).reshape(-1, L.Cin)[pix]
        prior = net.prior_of_input[L.name]
        if net.gated_input.get(L.name):
            # the pass wrote the lower layer's dZ: its ReLU gate and folded batch-norm scale are
            # applied to the gradient in the epilogue (`prior` is that layer's output)
            P = net.layers[L.src]
            sc = P.extra["scale"].cpu().numpy().astype(np.float64) if P.extra["scale"] is not None else np.ones(L.Cin)
            gate = f64(prior).reshape(-1, L.Cin)[pix] > 0
            ref = np.where(gate, ref * sc, 0.0)
            tol = tol * np.abs(sc)
        elif prior is not None:
            ref = ref + f64(prior).reshape(-1, L.Cin)[pix]
        within(got, ref, tol, True)


def record_dx(net):
    """Wraps conv2d_bwd_data to keep, per layer, a copy of what was in the output buffer before
    (the other branch's gradient) and of the result."""
    net.grad_of_input, net.prior_of_input, net.gated_input = {}, {}, {}
    orig = twn.conv2d_bwd_data
    by_desc = {id(L.desc): L for L in net.layers.values()}

    def wrapped(desc, dZ, T_bwd, ld, stats, epi, dX, status=None, stream=None):
        L = by_desc[id(desc)]
        prior = None
        if epi is not None and epi.residual:
            src = net.last_res
            prior = src.clone()
        orig(desc, dZ, T_bwd, ld, stats, epi, dX, status, stream)
        net.grad_of_input[L.name] = dX.clone()
        net.prior_of_input[L.name] = prior
        net.gated_input[L.name] = epi is not None and epi.residual_op == twn.RESIDUAL_GATE
    return orig, wrapped


def run_train_step(net, monkeypatch):
    x = dg.draw_bf16(0, f"{net.name}.input", net.act["input"].numel(), "normal")
    net.set_input(x)
    last = net.ops[-1][1]
    dy_bits = dg.draw_bf16(0, f"{net.name}.dlogits", net.B * last.Cout, "normal", 0.0, 0.1)
    dY = torch.from_numpy(dy_bits.view(np.int16)).cuda().view(torch.bfloat16).view(net.B, last.Cout)
    # keep copies of every backward-for-data result and of the residual it was added to
    orig_epi = twn.epilogue

    def epi_spy(scale=None, shift=None, residual=None, relu=False, out_dtype=twn.F32, residual_op=twn.RESIDUAL_ADD):
        net.last_res = residual
        return orig_epi(scale, shift, residual, relu, out_dtype, residual_op)
    orig, wrapped = record_dx(net)
    monkeypatch.setattr(twn, "epilogue", epi_spy)
    monkeypatch.setattr(twn, "conv2d_bwd_data", wrapped)
    net.train_step(dY)
    torch.cuda.synchronize()
    net.check_status()
    monkeypatch.setattr(twn, "conv2d_bwd_data", orig)
    monkeypatch.setattr(twn, "epilogue", orig_epi)


def test_lenet5_forward_batch100():
    net = nets.lenet5(100)
    net.set_input(dg.draw_bf16(0, "lenet5.input", 100 * 28 * 28, "uniform01"))
    net.ternarize_all()
    logits = net.forward()
    torch.cuda.synchronize()
    net.check_status()
    assert logits.shape == (100, 1, 1, 10) and logits.dtype == torch.float32
    check_forward(net, npix=400)
    check_pools(net, images=100)


def test_vgg7_forward_batch128():
    net = nets.vgg7(128)
    net.set_input(dg.draw_bf16(0, "vgg7.input", 128 * 32 * 32 * 3, "normal"))
    net.ternarize_all()
    logits = net.forward()
    torch.cuda.synchronize()
    net.check_status()
    assert logits.shape == (128, 1, 1, 10)
    check_forward(net)
    check_pools(net)


def test_resnet18_small_train_step(monkeypatch):
    net = nets.resnet18(batch=2, train=True, image=64, classes=24)
    run_train_step(net, monkeypatch)
    check_forward(net, npix=400)
    check_pools(net)
    check_backward(net, npix=300, nent=300)


def test_resnet18b_wider_stages_small_train_step(monkeypatch):
    """The 1.5x wider variant of the paper's ImageNet experiments: 96/192/384/768 channels, i.e.
    reductions that are not multiples of 64 per tap (the last 64-channel block of a tap is half
    empty and the code columns of a tap do not start on 16-byte boundaries)."""
    net = nets.resnet18b(batch=2, train=True, image=64, classes=24)
    run_train_step(net, monkeypatch)
    check_forward(net, npix=300)
    check_pools(net)
    check_backward(net, npix=200, nent=200)


def test_resnet18_small_steps_with_parameter_update():
    """Algorithm 1 end to end, twice: ternarize, forward, backward, SGD update.  The update is checked
    against the oracle on the GPU's own gradients (bit-exact), and the second step's codes, which come
    from the coding sweep alone with the thresholds the update left behind, against the oracle's
    ternarization of the updated weights."""
    opt = dict(lr=1e-3, momentum=0.9, weight_decay=1e-4)
    net = nets.resnet18(batch=2, train=True, image=64, classes=24, optimizer=opt)
    x = dg.draw_bf16(0, "sgdnet.input", net.act["input"].numel(), "normal")
    net.set_input(x)
    dy_bits = dg.draw_bf16(0, "sgdnet.dlogits", 2 * 24, "normal", 0.0, 0.1)
    dY = torch.from_numpy(dy_bits.view(np.int16)).cuda().view(torch.bfloat16).view(2, 24)
    W = {n: L.extra["W"].cpu().numpy().copy() for n, L in net.layers.items()}
    V = {n: np.zeros_like(w) for n, w in W.items()}
    for step in range(2):
        net.train_step(dY)
        torch.cuda.synchronize()
        net.check_status()
        for n, L in net.layers.items():
            if step == 1:
                # this step's codes came from the coding sweep alone
                st, codes = oracle.ternarize(W[n], net.delta_factor)
                got = twn.stats_to_host(L.extra["stats"])
                assert st.n_boundary == 0
                assert np.array_equal(L.extra["packed"].cpu().numpy().view(np.uint32),
                                      oracle.pack(codes.reshape(L.Cout, L.K), L.extra["ld"]))
                assert abs(got["alpha"] - st.alpha) <= 1e-12 * st.alpha
            dW = L.extra["dW"].cpu().numpy().reshape(W[n].shape)
            W[n], V[n] = oracle.sgd_update(W[n], dW, V[n], opt["lr"], opt["momentum"], opt["weight_decay"])
            assert np.array_equal(L.extra["W"].cpu().numpy().view(np.uint32), W[n].view(np.uint32))
            assert np.array_equal(L.extra["V"].cpu().numpy().view(np.uint32), V[n].view(np.uint32))
            # the threshold for the next step is already there
            st_next, _ = oracle.ternarize(W[n], net.delta_factor)
            got = twn.stats_to_host(L.extra["stats"])
            assert got["status"] == 0 and abs(got["delta"] - st_next.delta) <= 1e-12 * st_next.delta


def test_resnet18_train_step_batch64(monkeypatch):
    net = nets.resnet18(batch=64, train=True)
    run_train_step(net, monkeypatch)
    check_forward(net, npix=96)
    check_pools(net, images=1)
    check_backward(net, npix=64, nent=96)


def test_resnet18b_train_step_batch64(monkeypatch):
    """The wider variant at the size the benchmark runs it: batch 64, 224 x 224."""
    net = nets.resnet18b(batch=64, train=True)
    run_train_step(net, monkeypatch)
    check_forward(net, npix=64)
    check_pools(net, images=1)
    check_backward(net, npix=48, nent=64)
