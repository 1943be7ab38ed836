"""Per-head selection (Section 8.5) through the C ABI against the oracle run head by head
(needs a B200).  The oracle has no notion of heads: a head is a T x d_h sequence of its own."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03110_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TAU = 0.3


@pytest.fixture(scope="module")
def ada():
    from paper_2605_03110_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return binding


def clustered_heads(T, h, d_h, seed, dtype, noise=0.05):
    """T tokens x h heads; every head has its own T/5 prototypes and its own assignment of
    tokens to them, so the representative sets differ from head to head."""
    rng = np.random.default_rng(seed)
    P = max(1, T // 5)
    X = np.empty((T, h, d_h))
    for j in range(h):
        base = rng.standard_normal((P, d_h))
        X[:, j] = base[rng.integers(0, P, T)] + noise * rng.standard_normal((T, d_h))
        X[rng.integers(0, T, max(1, T // 10)), j] = rng.standard_normal((max(1, T // 10), d_h))
    X = X.astype(np.float32)
    return wl.f32_to_bf16_bits(X) if dtype == "bf16" else X


def perturbed(X, seed, scale=0.3):
    rng = np.random.default_rng(seed)
    if X.dtype == np.uint16:
        return wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(X) + scale * rng.standard_normal(X.shape).astype(np.float32))
    return X + scale * rng.standard_normal(X.shape).astype(np.float32)


@pytest.mark.parametrize("dtype,engine", [("bf16", 0), ("bf16", 1), ("bf16", 2), ("bf16", 3), ("f32", 0),
                                          ("f32", 1), ("f32", 3)])
# (150, 80, 64): more sequences than the kernel keeps sequence tables for
@pytest.mark.parametrize("T,h,d_h", [(1, 1, 8), (2, 3, 8), (129, 3, 72), (300, 8, 64), (600, 5, 128),
                                     (257, 2, 256), (150, 80, 64)])
def test_heads_small_shapes(ada, dtype, engine, T, h, d_h):
    from parity import check_cascade, check_full
    ctx = ada.ada_create(h, T, d_h, ada.ADA_F32 if dtype == "f32" else ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    X0 = clustered_heads(T, h, d_h, 77 + T + h + d_h, dtype)
    X1 = perturbed(X0, T * 3 + h)
    _, reps = check_full(ctx, X0, TAU, heads=True)
    assert len(reps) == h
    if T >= 129 and h > 1:
        assert len({tuple(r.tolist()) for r in reps}) > 1
    for causal in (False, True):
        check_cascade(ctx, X1, TAU, reps, causal=causal, heads=True)
    # different degenerate inherited sets in different heads
    deg = [[], list(range(T)), [T - 1]]
    check_cascade(ctx, X1, TAU, [deg[j % 3] for j in range(h)], heads=True)
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_heads_equal_stacked_sequences_bit_for_bit(ada, dtype):
    """The interleaved layout (with a padded row stride) gives exactly what the same heads give
    when they are copied out and stacked as sequences."""
    from parity import to_device
    T, h, d_h, pad = 700, 6, 64, 24
    X0 = clustered_heads(T, h, d_h, 5, dtype)
    X1 = perturbed(X0, 6)
    ctx = ada.ada_create(h, T, d_h, ada.ADA_F32 if dtype == "f32" else ada.ADA_BF16)
    outs = []
    for layout in ("heads", "stacked"):
        res = []
        R = None
        for Xnp in (X0, X1):
            Xd = to_device(Xnp)
            if layout == "heads":
                big = torch.zeros((T, h * d_h + pad), dtype=Xd.dtype, device="cuda")
                big[:, :h * d_h] = Xd.reshape(T, h * d_h)
                Xv = big[:, :h * d_h].unflatten(1, (h, d_h))
                assert Xv.stride() == (h * d_h + pad, d_h, 1)
                if R is None:
                    R = ada.ada_select_full_heads(ctx, Xv, TAU)
                    res += [R[0], R[1], R[2]]
                else:
                    o = ada.ada_cascade_step_heads(ctx, Xv, TAU, R[0], R[1])
            else:
                Xs = Xd.permute(1, 0, 2).contiguous()
                if R is None:
                    R = ada.ada_select_full(ctx, Xs, TAU)
                    res += [R[0], R[1], R[2]]
                else:
                    o = ada.ada_cascade_step(ctx, Xs, TAU, R[0], R[1])
        res += [o.rep_out, o.rep_out_cnt, o.add_idx, o.add_cnt, o.rem_idx, o.rem_cnt, o.gamma_rep,
                o.gamma_cross]
        outs.append([t.cpu() for t in res])
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    cnt = {1: outs[0][1], 4: outs[0][4], 6: outs[0][6], 8: outs[0][8]}
    for k, (a, b) in enumerate(zip(*outs)):
        if k + 1 in cnt:       # an index list: compare the filled part
            for j in range(h):
                n = int(cnt[k + 1][j])
                assert torch.equal(a[j, :n], b[j, :n])
        else:
            assert torch.equal(a, b), k
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("h,d_h", [(32, 128), (16, 256)])
def test_heads_on_gptj_shaped_layers(ada, h, d_h):
    """T = 2048, d = 4096 activations of the GPT-J-shaped workload read as h heads of width
    d_h; three layers, each head checked against the oracle with the oracle's inherited sets."""
    from parity import check_cascade, check_full
    cfg = wl.CONFIGS[3]
    assert h * d_h == cfg.d
    ctx = ada.ada_create(h, cfg.T, d_h, ada.ADA_BF16)
    band_total, R = 0, None
    for lb in wl.generate_layers(cfg, seed=0, n_layers=3):
        X = lb.X[0].reshape(cfg.T, h, d_h)
        if lb.layer == 0:
            band, reps = check_full(ctx, X, cfg.tau, heads=True)
            R = reps
        else:
            band, _, refs = check_cascade(ctx, X, cfg.tau, R, heads=True)
            R = [r.rep for r in refs]
        band_total += band
    assert band_total == 0      # no tolerance band was needed on this workload
    ada.ada_destroy(ctx)


def test_heads_error_paths(ada):
    ctx = ada.ada_create(4, 64, 64, ada.ADA_BF16)
    lib, vp = ada.lib(), None
    X = torch.randn(64, 4, 64, device="cuda").to(torch.bfloat16)
    idx = torch.zeros((8, 64), dtype=torch.int32, device="cuda")
    cnt = torch.zeros(8, dtype=torch.int32, device="cuda")

    def full(T, h, d_h, ldx):
        return lib.ada_select_full_heads(ctx.h, X.data_ptr(), T, h, d_h, ldx, ada.ADA_BF16, TAU,
                                         idx.data_ptr(), cnt.data_ptr(), vp, vp)
    assert full(64, 4, 64, 256) == 0
    assert full(64, 4, 64, 248) == 1        # row stride below h * d_h
    assert full(64, 4, 64, 128) == 1
    assert full(64, 4, 64, 257) == 2        # row stride not a multiple of 16 bytes
    assert full(64, 8, 32, 256) == 3        # more heads than the context was created for
    assert full(64, 2, 128, 256) == 3       # head wider than the context's maxd
    assert full(64, 4, 60, 256) == 2        # head width not a multiple of 16 bytes
    assert full(64, 0, 64, 256) == 1
    st = lib.ada_cascade_step_heads(ctx.h, X.data_ptr(), 64, 4, 64, 248, ada.ADA_BF16, TAU,
                                    idx.data_ptr(), cnt.data_ptr(), idx.data_ptr(), cnt.data_ptr(),
                                    idx.data_ptr(), cnt.data_ptr(), idx.data_ptr(), cnt.data_ptr(),
                                    vp, vp, 0, vp)
    assert st == 1
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    ada.ada_destroy(ctx)


def test_heads_on_long_sequence_past_the_tile_table(ada):
    """T = 8192 as 32 heads x 128: every CTA gets a few hundred tiles, far more than the 80 its
    shared-memory table holds, so most tiles are located by the on-the-fly search.  Two heads are
    checked in full against the oracle, full selection and one cascade step."""
    from parity import TOL, check_set, lists, to_device
    cfg = wl.CONFIGS[4]
    h, d_h, T = 32, cfg.d // 32, cfg.T
    tol = TOL["bf16"]
    thr = 1.0 - cfg.tau * cfg.tau
    gen = wl.generate_layers(cfg, seed=0, n_layers=2)
    X0, X1 = [lb.X[0].reshape(T, h, d_h) for lb in gen]
    ctx = ada.ada_create(h, T, d_h, ada.ADA_BF16)
    idx, cnt, gamma = ada.ada_select_full_heads(ctx, to_device(X0), cfg.tau)
    out = ada.ada_cascade_step_heads(ctx, to_device(X1), cfg.tau, idx, cnt)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    reps, reps1 = lists(idx, cnt), lists(out.rep_out, out.rep_out_cnt)
    g, gc, gr = gamma.cpu().numpy(), out.gamma_cross.cpu().numpy(), out.gamma_rep.cpu().numpy()
    for j in (0, 17):
        x0 = wl.as_f64(np.ascontiguousarray(X0[:, j]))
        ref_rep, ref_g = oracle.select_full(x0, cfg.tau)
        assert np.max(np.abs(g[j] - ref_g)) <= tol
        assert check_set(reps[j], ref_g, np.arange(T), thr, tol) == 0
        assert reps[j].tolist() == ref_rep.tolist()
        ref = oracle.cascade_step(wl.as_f64(np.ascontiguousarray(X1[:, j])), cfg.tau, ref_rep)
        g_rep_tok = np.zeros(T)
        g_rep_tok[ref_rep] = ref.gamma_rep
        assert np.max(np.abs(gr[j] - g_rep_tok)) <= tol
        assert np.max(np.abs(gc[j] - ref.gamma_cross)) <= tol
        assert reps1[j].tolist() == ref.rep.tolist()
    ada.ada_destroy(ctx)
