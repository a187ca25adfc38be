"""The packed layer record (codes + fp16 tables / (S, Z)) and the stack driver, through the C ABI, against the oracle."""
import os

import numpy as np
import pytest
import torch

import synth
from oracle import leanquant_oracle as O

pytestmark = pytest.mark.gpu

CODE_TOL, LOSS_TOL, CENT_TOL = 1e-3, 1e-3, 1e-4


@pytest.fixture(scope="module")
def lq():
    import paper_2407_10032_b200 as m
    from paper_2407_10032_b200 import build
    build.build(debug_bounds=os.environ.get("LQ_LIBRARY_VARIANT") == "debug")
    return m


@pytest.fixture(scope="module")
def h(lq):
    handle = lq.lq_create(0)
    yield handle
    lq.lq_destroy(handle)


def f64(t):
    return t.detach().double().cpu().numpy()


@pytest.mark.parametrize("r,c,bits", [(37, 200, 3), (64, 4096, 4), (5, 33, 2), (300, 1024, 4)])
def test_record_nonuniform_bit_exact(lq, h, r, c, bits):
    g = torch.Generator().manual_seed(r + c)
    codes = torch.randint(0, 1 << bits, (r, c), generator=g, dtype=torch.uint8)
    grid = torch.sort(torch.randn(r, 1 << bits, generator=g) * 0.03, dim=1).values
    cfg = lq.Config.make(grid="nonuniform", bits=bits)
    rec = lq.lq_pack_layer(h, cfg, codes.cuda(), grid=grid.cuda())
    lq.lq_sync_status(h)
    want = O.pack_layer(codes.numpy(), bits, grid=grid.numpy())
    assert np.array_equal(rec.cpu().numpy(), want)
    nbytes, bpw = lq.lq_pack_layer_bytes(cfg, r, c)
    assert nbytes == want.size and abs(bpw - O.record_bits_per_weight(bits, c)) < 1e-12
    back = lq.lq_unpack_layer(h, cfg, rec, r, c)
    lq.lq_sync_status(h)
    assert np.array_equal(f64(back), O.unpack_layer(want))


@pytest.mark.parametrize("r,c,bits,group", [(16, 512, 4, 128), (9, 384, 3, 64), (7, 256, 4, 0), (12, 96, 2, 32)])
def test_record_affine_bit_exact(lq, h, r, c, bits, group):
    g = torch.Generator().manual_seed(r * c)
    ng = 1 if group == 0 else c // group
    codes = torch.randint(0, 1 << bits, (r, c), generator=g, dtype=torch.uint8)
    scale = torch.rand(r, ng, generator=g) * 0.01 + 1e-4
    zero = torch.randint(-4, 1 << bits, (r, ng), generator=g, dtype=torch.int32)
    cfg = lq.Config.make(grid="affine", bits=bits, group=group, T=45, t=9)
    rec = lq.lq_pack_layer(h, cfg, codes.cuda(), scale=scale.cuda(), zero=zero.cuda())
    lq.lq_sync_status(h)
    want = O.pack_layer(codes.numpy(), bits, scale=scale.numpy(), zero=zero.numpy(), group=group)
    assert np.array_equal(rec.cpu().numpy(), want)
    assert abs(lq.lq_pack_layer_bytes(cfg, r, c)[1] - O.record_bits_per_weight(bits, c, "affine", group)) < 1e-12
    back = lq.lq_unpack_layer(h, cfg, rec, r, c)
    lq.lq_sync_status(h)
    assert np.array_equal(f64(back), O.unpack_layer(want))


def test_record_zero_point_out_of_range_is_reported(lq, h):
    codes = torch.zeros(2, 64, dtype=torch.uint8, device="cuda")
    scale = torch.ones(2, 1, device="cuda")
    zero = torch.tensor([[5], [70000]], dtype=torch.int32, device="cuda")
    cfg = lq.Config.make(grid="affine", bits=4, group=0, T=45, t=9)
    lq.lq_pack_layer(h, cfg, codes, scale=scale, zero=zero)
    st, info = lq.lq_sync_status(h, raise_on_error=False)
    assert st == 2 and info == 1


def test_stack_of_layers_sharing_hessians(lq, h):
    """A small decoder-block-shaped stack in order: q / k / v share one Hessian, o has its own, gate / up share one,
    down has its own.  Every layer against the oracle's pass on the same inputs; records against the oracle's packing
    of the library's own codes and grids; a dead input channel of a shared group is zeroed in all of its layers."""
    n, bits = 4096, 3
    spec = [(256, "c2", [256, 64, 64]), (256, "c2", [256]), (256, "c2", [640, 640]), (640, "c3", [256])]
    cfg = lq.Config.make(grid="nonuniform", bits=bits, p=4.0, n_iter=20)
    S = lq.StackPass(h, [(c, rs) for c, _, rs in spec], cfg, w_dtype=torch.float32, x_dtype=torch.bfloat16, n_chunk=n,
                     device="cuda", want_w_hat=True)
    inputs, weights, groups_o = [], [], []
    for gi, (c, recipe, rs) in enumerate(spec):
        X = synth.make_layer(recipe, 8, c, n, seed=100 + gi).X
        if gi == 0:
            X[17] = 0                                 # a channel that never fires, in the group that three layers share
        Ws = [synth.make_layer(recipe, r, c, 8, seed=200 + 10 * gi + li).W for li, r in enumerate(rs)]
        inputs.append(X.cuda())
        weights.append([W.cuda() for W in Ws])
        groups_o.append((f64(X), [f64(W) for W in Ws]))
    S.run(inputs, weights)
    lq.lq_sync_status(h)
    ref = O.run_stack(groups_o, bits=bits, p=4.0, block=128, n_iter=20)
    k = 0
    for gi, (c, recipe, rs) in enumerate(spec):
        for li, r in enumerate(rs):
            P, o = S.passes[gi][li], ref[k]
            k += 1
            W = groups_o[gi][1][li]
            if gi == 0:
                assert float(weights[gi][li][:, 17].abs().max()) == 0.0
            G = f64(P.grid)
            span = (W.max(1) - W.min(1))[:, None] / G.shape[1]
            rows_ok = np.all(np.abs(G - o["grid"]) <= CENT_TOL * np.maximum(np.abs(o["grid"]), span), axis=1)
            codes = P.codes.cpu().numpy().astype(np.int64)
            same = ~(codes != o["codes"]).any(axis=1)
            print(f"group {gi} layer {li} ({r} x {c}): {rows_ok.mean():.4f} of rows with the oracle's centroids, "
                  f"{(same & rows_ok).sum()} of {rows_ok.sum()} of them with the oracle's codes, "
                  f"loss rel err {abs(P.loss.item() / o['loss'] - 1):.1e}")
            # short rows (256 weights, 8 clusters, p = 4): a weight that sits on a midpoint to within the fp32 rounding of
            # the inverse diagonal may change sides and move a light centroid; such rows are few
            assert rows_ok.mean() >= 0.99
            assert (~same[rows_ok]).sum() <= max(2, 0.02 * r)
            assert abs(P.loss.item() / o["loss"] - 1) <= 5 * LOSS_TOL
            rec = S.records[gi][li].cpu().numpy()
            assert np.array_equal(rec, O.pack_layer(codes, bits, grid=f64(P.grid).astype(np.float32)))
            back = lq.lq_unpack_layer(h, cfg, S.records[gi][li], r, c)
            assert np.array_equal(f64(back), O.unpack_layer(rec))
    lq.lq_sync_status(h)
