"""GPU parity of the 3x3 convolution forward kernel (every node with the filters of its own parameter row)
against the convolution oracle, on the CIFAR-shaped layer family: 32x32x3 inputs, widths 16/32/64, stride 2
where the width doubles."""
import numpy as np
import pytest
import torch

from oracle import conv_oracle as co
from paper_1705_09056_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu

TOL_L2 = 1e-5        # per node, ||y - y_oracle|| / ||y_oracle||: products carry ~2^-21 each (three TF32 MMAs), K <= 576 terms
TOL_EL = 2e-5        # per element, relative to the largest |y| of the node (a missing tap would be ~1e-1)


def _context(params: torch.Tensor):
    n, N = params.shape
    ld = wl.padded_ld(N)
    X0 = torch.zeros((n, ld), device="cuda")
    X0[:, :N] = params.cuda()
    X1, G = torch.zeros_like(X0), torch.zeros_like(X0)
    ctx = binding.Dpsgd(n, N, *wl.ring(n), gamma=0.1)
    ctx.bind(X0, X1, G)
    return ctx


def _check(y_gpu: torch.Tensor, y_ref: np.ndarray, what):
    n = y_ref.shape[0]
    got = y_gpu.cpu().numpy().astype(np.float64).reshape(n, -1)
    ref = y_ref.reshape(n, -1)
    l2 = np.linalg.norm(got - ref, axis=1) / np.maximum(np.linalg.norm(ref, axis=1), 1e-30)
    el = np.abs(got - ref).max(axis=1) / np.maximum(np.abs(ref).max(axis=1), 1e-30)
    assert l2.max() <= TOL_L2 and el.max() <= TOL_EL, (what, float(l2.max()), float(el.max()))


def _offsets(plan):
    offs, off = [], 0
    for (cin, cout, _) in plan:
        offs.append((off, off + cout * cin * 9))
        off += cout * cin * 9 + cout
    return offs


@pytest.mark.parametrize("n,batch", [(3, 4), (2, 32), (5, 1)])
def test_cifar_layer_family_layer_by_layer_and_chained(n, batch):
    """Every layer of the family from the oracle's own (fp32) input activation, then the whole stack chained on
    the device.  batch = 1 leaves the last tile of the 8x8 layers half empty."""
    w = wl.conv_workload(n=n, batch=batch, seed=11)
    ctx = _context(w.params)
    acts = [co.layers_forward(w.inputs[i].numpy(), w.params[i].numpy(), w.plan) for i in range(n)]
    x_dev = w.inputs.cuda()
    chained = x_dev
    for l, ((cin, cout, stride), (w_off, b_off)) in enumerate(zip(w.plan, _offsets(w.plan))):
        x_l = torch.from_numpy(np.stack([acts[i][l] for i in range(n)])).cuda()
        y = ctx.conv3x3_forward(x_l, cout, stride, w_off, b_off, relu=True)
        ref = np.stack([acts[i][l + 1] for i in range(n)]).astype(np.float64)
        _check(y, ref, ("layer", l))
        chained = ctx.conv3x3_forward(chained, cout, stride, w_off, b_off, relu=True)
    ref = np.stack([acts[i][-1] for i in range(n)]).astype(np.float64)
    got = chained.cpu().numpy().astype(np.float64).reshape(n, -1)
    l2 = np.linalg.norm(got - ref.reshape(n, -1), axis=1) / np.linalg.norm(ref.reshape(n, -1), axis=1)
    assert l2.max() <= 1e-4, float(l2.max())          # six layers of rounding differences, ReLU is continuous
    ctx.sync()
    ctx.close()


@pytest.mark.parametrize("cin,cout,h,wd,stride,relu", [
    (5, 16, 8, 8, 1, False),      # K = 45: not a multiple of 8, filters at an odd offset (scalar loads)
    (16, 48, 16, 16, 2, True),    # three channel groups of 16
    (7, 32, 4, 32, 1, False),     # a 4 x 32 image is exactly one tile
    (4, 64, 64, 64, 2, True),     # 32 x 32 outputs from a 64 x 64 image
    (64, 64, 8, 8, 1, True),      # the widest layer: two launches over channel ranges
])
def test_other_shapes_without_relu_and_odd_offsets(cin, cout, h, wd, stride, relu):
    n, B = 3, 3
    rng = np.random.default_rng(cin * 100 + cout)
    pad = 3                                            # filters do not start on a 16-byte boundary
    N = pad + cout * cin * 9 + cout
    params = torch.zeros((n, N))
    params[:, pad:] = torch.from_numpy(rng.standard_normal((n, N - pad)).astype(np.float32) / np.sqrt(cin * 9))
    x = torch.from_numpy(rng.standard_normal((n, B, cin, h, wd)).astype(np.float32))
    ctx = _context(params)
    y = ctx.conv3x3_forward(x.cuda(), cout, stride, pad, pad + cout * cin * 9, relu=relu)
    ref = []
    for i in range(n):
        wi = params[i, pad:pad + cout * cin * 9].numpy().reshape(cout, cin, 3, 3)
        bi = params[i, pad + cout * cin * 9:].numpy()
        ref.append(co.conv3x3_forward(x[i].numpy(), wi, bi, stride, relu)[0])
    _check(y, np.stack(ref), (cin, cout, h, wd, stride))
    ctx.sync()
    ctx.close()


def test_filters_follow_the_current_parameter_buffer_and_bad_shapes_are_refused():
    """After a gossip step the layer reads X_{k+1}; unsupported shapes and blocks outside the row are errors."""
    w = wl.conv_workload(n=4, batch=2, seed=3)
    ctx = _context(w.params)
    (cin, cout, stride), (w_off, b_off) = w.plan[0], _offsets(w.plan)[0]
    x = w.inputs.cuda()
    before = ctx.conv3x3_forward(x, cout, stride, w_off, b_off)
    ctx.mix_update()                                   # G = 0: rows become ring averages of the filters
    after = ctx.conv3x3_forward(x, cout, stride, w_off, b_off)
    mixed = ctx.current()[:, :w.params.shape[1]].cpu().numpy()
    ref = np.stack([co.layers_forward(w.inputs[i].numpy(), mixed[i], w.plan)[1] for i in range(4)]).astype(np.float64)
    _check(after, ref, "after mixing")
    assert not torch.equal(before, after)
    for bad in [dict(c_out=10), dict(stride=3), dict(w_off=w.params.shape[1])]:
        kw = dict(c_out=cout, stride=stride, w_off=w_off, b_off=b_off)
        kw.update(bad)
        with pytest.raises(binding.DpsgdError) as e:
            ctx.conv3x3_forward(x, kw["c_out"], kw["stride"], kw["w_off"], kw["b_off"])
        assert e.value.status in (binding.ERR_UNSUPPORTED, binding.ERR_ARG)
    with pytest.raises(binding.DpsgdError) as e:
        ctx.conv3x3_forward(torch.zeros((4, 2, 3, 24, 24), device="cuda"), 16, 1, w_off, b_off)   # width not a power of two
    assert e.value.status == binding.ERR_UNSUPPORTED
    ctx.sync()
    ctx.close()


def _backward_reference(x, params, w_off, b_off, cin, cout, stride, relu, dy):
    """Oracle: (dw, db, dx) of one node's layer, sums over the minibatch."""
    w = params[w_off:w_off + cout * cin * 9].reshape(cout, cin, 3, 3)
    b = params[b_off:b_off + cout]
    _, pre = co.conv3x3_forward(x, w, b, stride, relu)
    d = co.relu_backward(dy, pre) if relu else np.asarray(dy, dtype=np.float64)
    dw, db = co.conv3x3_weight_grad(d, x, stride)
    dx = co.conv3x3_input_grad(d, w, x.shape[2:], stride)
    return dw, db, dx


@pytest.mark.parametrize("n,batch", [(3, 4), (2, 16)])
def test_backward_of_every_cifar_layer_matches_the_oracle(n, batch):
    """Filter, bias and input gradients of each layer of the family, from the oracle's activations and a random
    gradient at the layer's output.  The first layer (3 input channels) needs no input gradient."""
    w = wl.conv_workload(n=n, batch=batch, seed=12)
    ctx = _context(w.params)
    Gdev = ctx._keep[2]
    rng = np.random.default_rng(batch)
    acts = [co.layers_forward(w.inputs[i].numpy(), w.params[i].numpy(), w.plan) for i in range(n)]
    for l, ((cin, cout, stride), (w_off, b_off)) in enumerate(zip(w.plan, _offsets(w.plan))):
        x_l = np.stack([acts[i][l] for i in range(n)])
        y_l = np.stack([acts[i][l + 1] for i in range(n)])
        dy = rng.standard_normal(y_l.shape).astype(np.float32)
        Gdev.fill_(7.0)
        want_dx = cin % 16 == 0
        dx = ctx.conv3x3_backward(torch.from_numpy(x_l).cuda(), torch.from_numpy(y_l).cuda(), torch.from_numpy(dy).cuda(),
                                  stride, w_off, b_off, relu=True, want_dx=want_dx)
        G = Gdev.cpu().numpy().astype(np.float64)
        refs = [_backward_reference(x_l[i], w.params[i].numpy(), w_off, b_off, cin, cout, stride, True, dy[i]) for i in range(n)]
        dw = G[:, w_off:w_off + cout * cin * 9]
        db = G[:, b_off:b_off + cout]
        dw_ref = np.stack([r[0].reshape(-1) for r in refs])
        db_ref = np.stack([r[1] for r in refs])
        assert np.linalg.norm(dw - dw_ref, axis=1).max() <= 1e-5 * np.linalg.norm(dw_ref, axis=1).min(), ("dw", l)
        assert np.abs(dw - dw_ref).max() <= 2e-5 * np.abs(dw_ref).max(), ("dw", l)
        assert np.abs(db - db_ref).max() <= 2e-5 * np.abs(db_ref).max() + 1e-6, ("db", l)
        # nothing but the layer's own blocks of G is written
        keep = np.ones(G.shape[1], dtype=bool)
        keep[w_off:w_off + cout * cin * 9] = False
        keep[b_off:b_off + cout] = False
        assert np.all(G[:, keep] == 7.0), l
        if want_dx:
            _check(dx, np.stack([r[2] for r in refs]), ("dx", l))
    ctx.sync()
    ctx.close()


def test_backward_without_relu_ragged_batch_and_refusals():
    n, B, cin, cout, h, wd, stride = 2, 3, 16, 32, 8, 8, 2
    rng = np.random.default_rng(9)
    N = cout * cin * 9 + cout
    params = torch.from_numpy(rng.standard_normal((n, N)).astype(np.float32) / np.sqrt(cin * 9))
    x = rng.standard_normal((n, B, cin, h, wd)).astype(np.float32)
    dy = rng.standard_normal((n, B, cout, 4, 4)).astype(np.float32)
    ctx = _context(params)
    dx = ctx.conv3x3_backward(torch.from_numpy(x).cuda(), None, torch.from_numpy(dy).cuda(), stride, 0, cout * cin * 9,
                              relu=False)
    G = ctx._keep[2].cpu().numpy().astype(np.float64)
    refs = [_backward_reference(x[i], params[i].numpy(), 0, cout * cin * 9, cin, cout, stride, False, dy[i]) for i in range(n)]
    dw_ref = np.stack([r[0].reshape(-1) for r in refs])
    assert np.abs(G[:, :cout * cin * 9] - dw_ref).max() <= 2e-5 * np.abs(dw_ref).max()
    assert np.abs(G[:, cout * cin * 9:N] - np.stack([r[1] for r in refs])).max() <= 2e-5 * np.abs(dw_ref).max()
    _check(dx, np.stack([r[2] for r in refs]), "dx without relu")
    with pytest.raises(binding.DpsgdError) as e:           # a ReLU layer needs its output for the mask
        ctx.conv3x3_backward(torch.from_numpy(x).cuda(), None, torch.from_numpy(dy).cuda(), stride, 0, cout * cin * 9, relu=True)
    assert e.value.status == binding.ERR_ARG
    with pytest.raises(binding.DpsgdError) as e:           # filters outside the row
        ctx.conv3x3_backward(torch.from_numpy(x).cuda(), None, torch.from_numpy(dy).cuda(), stride, cout + 1, cout * cin * 9, relu=False)
    assert e.value.status == binding.ERR_ARG
    ctx.sync()
    ctx.close()
