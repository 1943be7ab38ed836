"""GPU-vs-oracle parity of the selection path, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03110_b200 import workloads as wl
from label_model import cascade_from_labels, full_from_labels

pytestmark = pytest.mark.gpu

TAU = 0.3


@pytest.fixture(scope="module")
def ada():
    from paper_2605_03110_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return binding


def clustered(T, d, seed, dtype):
    rng = np.random.default_rng(seed)
    P = max(1, T // 5)
    base = rng.standard_normal((P, d))
    X = base[rng.integers(0, P, T)] + 0.05 * rng.standard_normal((T, d))
    X[rng.integers(0, T, max(1, T // 10))] = rng.standard_normal((max(1, T // 10), d))
    X = X.astype(np.float32)[None]
    return wl.f32_to_bf16_bits(X) if dtype == "bf16" else X


# (storage, engine): 0 AUTO, 1 forced FFMA, 2 forced one-CTA tcgen05, 3 forced pair-CTA tcgen05
# (fp32 storage reaches the tensor cores through the three-term bf16 split)
ENGINES = [("f32", 0), ("f32", 1), ("f32", 3), ("bf16", 0), ("bf16", 1), ("bf16", 2), ("bf16", 3)]


@pytest.mark.parametrize("dtype,engine", ENGINES)
@pytest.mark.parametrize("T", [1, 2, 3, 127, 128, 129, 257, 600])
@pytest.mark.parametrize("d", [8, 72, 768])
def test_small_shapes_full_and_cascade(ada, dtype, engine, T, d):
    from parity import check_cascade, check_full
    ctx = ada.ada_create(1, T, d, ada.ADA_F32 if dtype == "f32" else ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    X0 = clustered(T, d, 1000 + T + d, dtype)
    X1 = clustered(T, d, 1000 + T + d, dtype)       # same prototypes, then perturbed
    rng = np.random.default_rng(T * 7 + d)
    if dtype == "bf16":
        X1 = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(X1) + 0.3 * rng.standard_normal(X1.shape).astype(np.float32))
    else:
        X1 = X1 + 0.3 * rng.standard_normal(X1.shape).astype(np.float32)
    # the checks assert parity outside the tolerance band; at tiny d a gamma may
    # land inside it by chance, which is tolerated (and counted) by design
    band, reps = check_full(ctx, X0, TAU)
    for causal in (False, True):
        check_cascade(ctx, X1, TAU, reps, causal=causal)
    # degenerate inherited sets: empty, everything, a single token
    for R in ([], list(range(T)), [T - 1]):
        check_cascade(ctx, X1, TAU, [R])
    ada.ada_destroy(ctx)


def run_config_chain(ada, cfg, n_layers=None, causal=False, engine=0):
    """Step parity with the oracle chain's inherited sets fed to both sides,
    plus the free-running GPU chain (its own sets fed forward)."""
    from parity import check_cascade, check_full, lists, to_device
    ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_F32 if cfg.dtype == "f32" else ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    band_total = 0
    R_oracle = None
    free_idx = free_cnt = None
    for lb in wl.generate_layers(cfg, seed=0, n_layers=n_layers):
        Xd = to_device(lb.X)
        if lb.layer == 0:
            band, reps = check_full(ctx, lb.X, cfg.tau)
            R_oracle = reps if band == 0 else [oracle.select_full(wl.as_f64(lb.X[b]), cfg.tau)[0]
                                               for b in range(cfg.B)]
            free_idx, free_cnt, _ = ada.ada_select_full(ctx, Xd, cfg.tau)
        else:
            band, _, refs = check_cascade(ctx, lb.X, cfg.tau, R_oracle, causal=causal)
            R_oracle = [r.rep for r in refs]
            out = ada.ada_cascade_step(ctx, Xd, cfg.tau, free_idx, free_cnt,
                                       flags=ada.ADA_CROSS_CAUSAL if causal else 0)
            free_idx, free_cnt = out.rep_out, out.rep_out_cnt
        band_total += band
        for b in range(cfg.B):      # label-level prediction of the full selection (no Gram)
            assert full_from_labels(lb.labels[b]).tolist() == \
                oracle.select_full(wl.as_f64(lb.X[b]), cfg.tau)[0].tolist() or cfg.T > 4096
    if band_total == 0:
        free = lists(free_idx, free_cnt)
        for b in range(cfg.B):
            assert free[b].tolist() == R_oracle[b].tolist()
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    ada.ada_destroy(ctx)
    return band_total


@pytest.mark.parametrize("engine", [0, 1])
def test_config1_gpt2_shaped_fp32(ada, engine):
    assert run_config_chain(ada, wl.CONFIGS[1], engine=engine) == 0


@pytest.mark.parametrize("causal", [False, True])
def test_config2_batched_bf16(ada, causal):
    assert run_config_chain(ada, wl.CONFIGS[2], n_layers=6, causal=causal) == 0


def test_config3_gptj_shaped_bf16(ada):
    assert run_config_chain(ada, wl.CONFIGS[3], n_layers=5) == 0


def test_config2_ffma_engine_matches(ada):
    assert run_config_chain(ada, wl.scaled(wl.CONFIGS[2], B=2), n_layers=3, engine=1) == 0


@pytest.mark.parametrize("engine", [2, 3])
def test_config2_and_3_on_both_tensor_core_kernels(ada, engine):
    assert run_config_chain(ada, wl.CONFIGS[2], n_layers=4, causal=True, engine=engine) == 0
    assert run_config_chain(ada, wl.CONFIGS[3], n_layers=4, engine=engine) == 0


def sampled_large(ada, cfg, n_layers, n_sample=48, engine=0, per_tile=False):
    """Full-size check where the oracle cannot do a whole layer quickly: sets by the
    label-level prediction (exact, no Gram), gamma on sampled rows by the oracle."""
    from parity import TOL, lists, to_device
    tol = TOL[cfg.dtype]
    ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    rng = np.random.default_rng(5)
    R_lab = None
    for lb in wl.generate_layers(cfg, seed=0, n_layers=n_layers):
        Xd = to_device(lb.X)
        lab = lb.labels[0]
        X64 = wl.as_f64(lb.X[0])
        rep_idx, rep_cnt, gamma = ada.ada_select_full(ctx, Xd, cfg.tau)
        full = lists(rep_idx, rep_cnt)[0]
        assert full.tolist() == full_from_labels(lab).tolist()
        rows = tile_rows(rng, cfg.T, n_sample) if per_tile else \
            np.sort(rng.choice(cfg.T, n_sample, replace=False)).astype(np.int32)
        g_ref = oracle.full_rows(X64, rows)
        assert np.max(np.abs(gamma.cpu().numpy()[0][rows] - g_ref)) <= tol
        if lb.layer == 0:
            R_lab = full
            R_idx, R_cnt = rep_idx, rep_cnt
            continue
        out = ada.ada_cascade_step(ctx, Xd, cfg.tau, R_idx, R_cnt)
        exp_rep, exp_add, exp_rem = cascade_from_labels(lab, R_lab)
        assert lists(out.rep_out, out.rep_out_cnt)[0].tolist() == exp_rep.tolist()
        assert lists(out.add_idx, out.add_cnt)[0].tolist() == exp_add.tolist()
        assert lists(out.rem_idx, out.rem_cnt)[0].tolist() == exp_rem.tolist()
        nonrep = np.setdiff1d(np.arange(cfg.T), R_lab)
        if per_tile:
            rows = np.setdiff1d(tile_rows(rng, cfg.T, 2 * n_sample), R_lab).astype(np.int32)
        else:
            rows = np.sort(rng.choice(nonrep, min(n_sample, nonrep.size), replace=False)).astype(np.int32)
        ref = oracle.cascade_step(X64, cfg.tau, R_lab, only_rows=rows)
        assert np.max(np.abs(out.gamma_cross.cpu().numpy()[0][rows] - ref.gamma_cross[rows])) <= tol
        g_rep_tok = np.zeros(cfg.T)
        g_rep_tok[R_lab] = ref.gamma_rep
        assert np.max(np.abs(out.gamma_rep.cpu().numpy()[0] - g_rep_tok)) <= tol
        assert lists(out.rem_idx, out.rem_cnt)[0].tolist() == ref.rem.tolist()
        R_lab, R_idx, R_cnt = exp_rep, out.rep_out, out.rep_out_cnt
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("engine", [2, 3])
def test_config4_opt_shaped_full_size_sampled(ada, engine):
    sampled_large(ada, wl.CONFIGS[4], n_layers=3, engine=engine)


def elementwise_transition(ada, cfg, engine=0, causal=False):
    """Layer 0 -> layer 1 of `cfg` against the oracle in full: every gamma of the full selection,
    every gamma_rep and gamma_cross of the cascade step, sets and lists (both sides start the
    step from the oracle's set)."""
    from parity import check_cascade, check_full
    ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    band = 0
    R = None
    for lb in wl.generate_layers(cfg, seed=0, n_layers=2):
        if lb.layer == 0:
            b0, R = check_full(ctx, lb.X, cfg.tau)
            band += b0
            assert b0 == 0      # the workloads keep every gamma far from the threshold
            for b in range(cfg.B):
                assert R[b].tolist() == full_from_labels(lb.labels[b]).tolist()
        else:
            b1, _, _ = check_cascade(ctx, lb.X, cfg.tau, R, causal=causal)
            band += b1
    assert ada.ada_device_status(ctx)[0] == 0
    ada.ada_destroy(ctx)
    return band


@pytest.mark.parametrize("engine", [0, 3])
def test_config4_opt_shaped_full_size_elementwise(ada, engine):
    """configs[3] at full size (T = 8192, d = 4096): one full selection and one cascade step,
    all 8192 gamma / gamma_rep / gamma_cross values and every list against the oracle."""
    assert elementwise_transition(ada, wl.CONFIGS[4], engine=engine) == 0


def test_config4_late_layer_cascade_step_elementwise(ada):
    """A cascade step of configs[3] with a late layer's large inherited set (three rounds of
    tiles on the pair kernel): the inherited set comes from the label-level replay of the
    chain (no Gram), the step itself is compared with the oracle element by element."""
    from parity import check_cascade
    cfg = wl.CONFIGS[4]
    n_layers = 24
    R = None
    for lb in wl.generate_layers(cfg, seed=0, n_layers=n_layers):
        if lb.layer == 0:
            R = full_from_labels(lb.labels[0])
        elif lb.layer < n_layers - 1:
            R = cascade_from_labels(lb.labels[0], R)[0]
        else:
            assert len(R) > 1024
            ctx = ada.ada_create(1, cfg.T, cfg.d, ada.ADA_BF16)
            band, rep, _ = check_cascade(ctx, lb.X, cfg.tau, [R])
            assert band == 0
            assert rep[0].tolist() == cascade_from_labels(lb.labels[0], R)[0].tolist()
            assert ada.ada_device_status(ctx)[0] == 0
            ada.ada_destroy(ctx)


def tile_rows(rng, T, n_sample, tile=128):
    """At least n_sample distinct rows, at least one from every `tile`-row block."""
    n_tiles = (T + tile - 1) // tile
    per = max(1, -(-n_sample // n_tiles))
    rows = []
    for i in range(n_tiles):
        lo, hi = i * tile, min(T, (i + 1) * tile)
        rows.extend(rng.choice(np.arange(lo, hi), min(per, hi - lo), replace=False).tolist())
    return np.sort(np.asarray(rows, dtype=np.int32))


# configs[4], the crossover sweep: every (T, r/T) point.  The oracle does whole layers up to
# T = 8192 and at the two extreme points of T = 16384; the two middle points of T = 16384 are
# checked by the label-level replay (sets) and the oracle on 512 rows, every 128-row tile hit.
SWEEP_FULL = [(T, q) for T in wl.SWEEP_T for q in wl.SWEEP_Q if T <= 8192 or q in (0.01, 0.5)]
SWEEP_SAMPLED = [(T, q) for T in wl.SWEEP_T for q in wl.SWEEP_Q if (T, q) not in SWEEP_FULL]


@pytest.mark.parametrize("T,q", SWEEP_FULL)
def test_sweep_points_elementwise(ada, T, q):
    assert elementwise_transition(ada, wl.sweep_config(T, q)) == 0


@pytest.mark.parametrize("T,q", SWEEP_SAMPLED)
def test_sweep_points_sampled(ada, T, q):
    sampled_large(ada, wl.sweep_config(T, q), n_layers=2, n_sample=512, per_tile=True)


def test_threshold_band_adversarial(ada):
    """Pairs built at cos = thr +- eps by a planar rotation embedded in d dims:
    outside the tolerance the decision must match; inside it either answer is
    accepted and counted."""
    from parity import check_full
    d, thr = 256, 1 - TAU * TAU
    for dtype, tol in (("f32", 1e-5), ("bf16", 2e-3)):
        ctx = ada.ada_create(1, 64, d, ada.ADA_F32 if dtype == "f32" else ada.ADA_BF16)
        rows = []
        rng = np.random.default_rng(11)
        Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
        k = 0
        for eps in (1e-2, 1e-3, 1e-4, 1e-6):
            for sgn in (+1, -1):
                theta = np.arccos(thr + sgn * eps)
                a, b = Q[2 * k], Q[2 * k + 1]
                rows.append(3.0 * a)
                rows.append(0.7 * (np.cos(theta) * a + np.sin(theta) * b))
                k += 1
        X = np.asarray(rows, dtype=np.float32)[None]
        Xs = wl.f32_to_bf16_bits(X) if dtype == "bf16" else X
        band, reps = check_full(ctx, Xs, TAU)      # asserts gamma within tol, sets outside the band
        _, g = oracle.select_full(wl.as_f64(Xs[0]), TAU)
        n_in_band = int(np.sum(np.abs(g - thr) <= tol))
        assert band <= n_in_band
        ada.ada_destroy(ctx)


def test_duplicates_orthogonal_and_zero_rows(ada):
    from parity import check_full, to_device
    d = 64
    Q, _ = np.linalg.qr(np.random.default_rng(2).standard_normal((d, d)))
    X = (Q[:40] * np.linspace(0.5, 4, 40)[:, None]).astype(np.float32)
    X[13] = -2.0 * X[4]
    X[29] = 0.0
    ctx = ada.ada_create(1, 40, d, ada.ADA_F32)
    band, reps = check_full(ctx, X[None], TAU)
    assert band == 0 and reps[0].tolist() == [t for t in range(40) if t != 13]
    ada.ada_select_full(ctx, to_device(X[None]), TAU)
    st, nz = ada.ada_device_status(ctx)
    assert st == 0 and nz == 1
    ada.ada_destroy(ctx)


def test_normalize_and_gather(ada):
    from parity import to_device
    cfg = wl.scaled(wl.CONFIGS[2], B=2, T=300, d=264, L=1)
    X = next(wl.generate_layers(cfg)).X
    Xd = to_device(X)
    ctx = ada.ada_create(2, 300, 264, ada.ADA_BF16)
    rep = np.zeros((2, 300), dtype=np.int32)
    rep[0, :4] = [0, 7, 8, 299]
    rep[1, :2] = [5, 100]
    cnt = np.array([4, 2], dtype=np.int32)
    inv, xhat, xrep = ada.ada_normalize(ctx, Xd, want_xhat=True, rep_idx=torch.from_numpy(rep).cuda(),
                                        rep_cnt=torch.from_numpy(cnt).cuda())
    for b in range(2):
        X64 = wl.as_f64(X[b])
        Xh, nrm = oracle.normalize(X64)
        assert np.allclose(inv[b].cpu().numpy() * nrm, 1.0, atol=1e-6)
        assert np.max(np.abs(xhat[b].float().cpu().numpy() - Xh)) <= 2.0 ** -8 * np.max(np.abs(Xh))
        got = xrep[b, :cnt[b]].view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got, X[b][rep[b, :cnt[b]]])
    ada.ada_destroy(ctx)


def test_error_paths(ada):
    from parity import to_device
    ctx = ada.ada_create(1, 64, 32, ada.ADA_F32)
    X = torch.randn(1, 64, 32, device="cuda")
    for tau in (0.0, 1.0, -0.3, float("nan")):
        with pytest.raises(ada.AdaError) as e:
            ada.ada_select_full(ctx, X, tau)
        assert e.value.status == 1
    with pytest.raises(ada.AdaError) as e:                      # above the context maxima
        ada.ada_select_full(ctx, torch.randn(1, 65, 32, device="cuda"), TAU)
    assert e.value.status == 3
    with pytest.raises(ada.AdaError) as e:                      # wrong storage type
        ada.ada_select_full(ctx, X.bfloat16(), TAU)
    assert e.value.status == 2
    with pytest.raises(ada.AdaError) as e:                      # d*es not a multiple of 16
        ada.ada_select_full(ctx, torch.randn(1, 64, 30, device="cuda"), TAU)
    assert e.value.status == 2
    flat = torch.randn(64 * 32 + 8, device="cuda")              # X not 16-byte aligned
    with pytest.raises(ada.AdaError) as e:
        ada.ada_select_full(ctx, flat[1:1 + 64 * 32].view(1, 64, 32), TAU)
    assert e.value.status == 2
    idx = torch.zeros((1, 64), dtype=torch.int32, device="cuda")
    cnt = torch.ones(1, dtype=torch.int32, device="cuda")
    with pytest.raises(ada.AdaError) as e:                      # rep_out must not alias rep_in
        out = ada.CascadeOut(1, 64, "cuda", False)
        out.rep_out = idx
        ada.ada_cascade_step(ctx, X, TAU, idx, cnt, out=out)
    assert e.value.status == 1
    with pytest.raises(ada.AdaError) as e:                      # unknown flag bit
        ada.ada_cascade_step(ctx, X, TAU, idx, cnt, flags=4)
    assert e.value.status == 1
    # host-buffer calls: storage type and alignment are checked before anything is copied
    hx = torch.randn(1, 64, 32).pin_memory()
    hi, hc = torch.empty(1, 64, dtype=torch.int32), torch.empty(1, dtype=torch.int32)
    with pytest.raises(ada.AdaError) as e:
        ada.ada_select_full_host(ctx, hx.bfloat16(), TAU, hi, hc)
    assert e.value.status == 2
    with pytest.raises(ada.AdaError) as e:
        ada.ada_cascade_step_host(ctx, hx.bfloat16(), TAU, hi, hc, hi.clone(), hc.clone(), hi.clone(),
                                  hc.clone(), hi.clone(), hc.clone())
    assert e.value.status == 2
    with pytest.raises(ada.AdaError) as e:
        ada.ada_select_full_host(ctx, torch.randn(1, 64, 30), TAU, hi, hc)
    assert e.value.status == 2
    # device-detected: unsorted inherited list, count out of range, NaN
    bad = torch.tensor([[3, 2] + [0] * 62], dtype=torch.int32, device="cuda")
    ada.ada_cascade_step(ctx, X, TAU, bad, torch.tensor([2], dtype=torch.int32, device="cuda"))
    assert ada.ada_device_status(ctx)[0] == 5
    ada.ada_cascade_step(ctx, X, TAU, bad, torch.tensor([65], dtype=torch.int32, device="cuda"))
    assert ada.ada_device_status(ctx)[0] == 5
    Xn = X.clone()
    Xn[0, 3, 3] = float("nan")
    ada.ada_select_full(ctx, Xn, TAU)
    assert ada.ada_device_status(ctx)[0] == 6
    ada.ada_select_full(ctx, X, TAU)                            # the context stays usable
    assert ada.ada_device_status(ctx)[0] == 0
    ada.ada_destroy(ctx)


def check_nearest(ada, ctx, Xnp, rep_lists, tol):
    """ada_nearest_rep vs the oracle: same index, except where the oracle's runner-up is within
    the tolerance of its maximum (then any representative that close is accepted)."""
    from parity import to_device
    B, T, _ = Xnp.shape
    rin = np.zeros((B, T), dtype=np.int32)
    rcnt = np.zeros(B, dtype=np.int32)
    for b, r in enumerate(rep_lists):
        rin[b, :len(r)] = r
        rcnt[b] = len(r)
    near, g = ada.ada_nearest_rep(ctx, to_device(Xnp), torch.from_numpy(rin).cuda(),
                                  torch.from_numpy(rcnt).cuda())
    assert ada.ada_device_status(ctx)[0] == 0
    near, g = near.cpu().numpy(), g.cpu().numpy()
    n_close = 0
    for b in range(B):
        X64 = wl.as_f64(Xnp[b])
        ref, gref = oracle.nearest(X64, rep_lists[b])
        assert np.max(np.abs(g[b] - gref), initial=0.0) <= tol
        diff = np.nonzero(near[b] != ref)[0]
        if diff.size:
            Xh, _ = oracle.normalize(X64)
            for t in diff:
                assert near[b][t] in set(rep_lists[b])
                assert abs(float(Xh[t] @ Xh[near[b][t]])) >= gref[t] - tol, (b, int(t))
                n_close += 1
    return n_close


@pytest.mark.parametrize("dtype,T,d", [("bf16", 1, 8), ("bf16", 300, 72), ("bf16", 1500, 512),
                                       ("f32", 129, 8), ("f32", 700, 256)])
def test_nearest_representative_small(ada, dtype, T, d):
    tol = 2e-3 if dtype == "bf16" else 1e-5
    ctx = ada.ada_create(1, T, d, ada.ADA_BF16 if dtype == "bf16" else ada.ADA_F32)
    X = clustered(T, d, 77 + T, dtype)
    full, _ = oracle.select_full(wl.as_f64(X[0]), TAU)
    for R in (full.tolist(), [], [T - 1], list(range(T)), list(range(0, T, 3))):
        check_nearest(ada, ctx, X, [R], tol)
    ada.ada_destroy(ctx)


def test_nearest_representative_on_configs(ada):
    """After full selection and after a cascade step, batched and at d = 4096."""
    from parity import lists, to_device
    for cfg, n_layers in ((wl.CONFIGS[2], 2), (wl.CONFIGS[3], 2)):
        ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_BF16)
        idx = cnt = None
        for lb in wl.generate_layers(cfg, seed=0, n_layers=n_layers):
            Xd = to_device(lb.X)
            if lb.layer == 0:
                idx, cnt, _ = ada.ada_select_full(ctx, Xd, cfg.tau)
            else:
                out = ada.ada_cascade_step(ctx, Xd, cfg.tau, idx, cnt)
                idx, cnt = out.rep_out, out.rep_out_cnt
            reps = [r.tolist() for r in lists(idx, cnt)]
            check_nearest(ada, ctx, lb.X, reps, 2e-3)
            near, _ = ada.ada_nearest_rep(ctx, Xd, idx, cnt)
            near = near.cpu().numpy()
            for b in range(cfg.B):          # label-level: the nearest representative shares the label
                nonrep = np.setdiff1d(np.arange(cfg.T), reps[b])
                assert np.all(lb.labels[b][near[b][nonrep]] == lb.labels[b][nonrep])
        # the workspace is clean again: a following selection is unaffected
        again = ada.ada_select_full(ctx, Xd, cfg.tau)
        ref = [oracle.select_full(wl.as_f64(lb.X[b]), cfg.tau)[0].tolist() for b in range(cfg.B)]
        assert [r.tolist() for r in lists(again[0], again[1])] == ref
        ada.ada_destroy(ctx)


@pytest.mark.parametrize("cfg_id,n_layers,causal", [(1, 12, False), (2, 12, True), (3, 28, False),
                                                    (3, 28, True), (4, 10, False)])
def test_full_length_free_running_chains_match_label_prediction(ada, cfg_id, n_layers, causal):
    """The production pattern at full size and depth: every layer's output set feeds the next
    call on the device, nothing is read back in between; the sets, additions and removals of
    every layer must equal the label-level replay of Definition 1 / Algorithm 1 (which uses
    no Gram at all)."""
    from parity import lists, to_device
    cfg = wl.CONFIGS[cfg_id]
    ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_F32 if cfg.dtype == "f32" else ada.ADA_BF16)
    flags = ada.ADA_CROSS_CAUSAL if causal else 0
    idx = cnt = None
    expect = [None] * cfg.B
    outs = []
    for lb in wl.generate_layers(cfg, seed=0, n_layers=n_layers):
        Xd = to_device(lb.X)
        if lb.layer == 0:
            idx, cnt, _ = ada.ada_select_full(ctx, Xd, cfg.tau, want_gamma=False)
            for b in range(cfg.B):
                expect[b] = (full_from_labels(lb.labels[b]), None, None)
            outs.append((idx.clone(), cnt.clone(), None))
        else:
            out = ada.ada_cascade_step(ctx, Xd, cfg.tau, idx, cnt, flags=flags, want_gamma=False)
            idx, cnt = out.rep_out, out.rep_out_cnt
            for b in range(cfg.B):
                expect[b] = cascade_from_labels(lb.labels[b], expect[b][0], causal)
            outs.append((idx.clone(), cnt.clone(),
                         (out.add_idx.clone(), out.add_cnt.clone(), out.rem_idx.clone(), out.rem_cnt.clone())))
        got = lists(*outs[-1][:2])
        for b in range(cfg.B):
            assert got[b].tolist() == expect[b][0].tolist(), (lb.layer, b)
            if lb.layer > 0:
                a_i, a_c, m_i, m_c = outs[-1][2]
                assert lists(a_i, a_c)[b].tolist() == expect[b][1].tolist()
                assert lists(m_i, m_c)[b].tolist() == expect[b][2].tolist()
    assert ada.ada_device_status(ctx)[0] == 0
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_padded_row_stride(ada, dtype):
    """ldx > d: X is a column slice of a wider buffer (TMA strides, vector loads, split kernel)."""
    from parity import lists
    T, d, ldx = 333, 200, 264
    X = clustered(T, d, 5, dtype)[0]
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    wide = torch.full((1, T, ldx), 7.0, dtype=tdt, device="cuda")          # padding must be ignored
    if dtype == "bf16":
        wide[0, :, :d] = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).cuda()
    else:
        wide[0, :, :d] = torch.from_numpy(X).cuda()
    Xv = wide[:, :, :d]
    assert Xv.stride(1) == ldx
    ctx = ada.ada_create(1, T, d, ada.ADA_BF16 if dtype == "bf16" else ada.ADA_F32)
    idx, cnt, gamma = ada.ada_select_full(ctx, Xv, TAU)
    ref_rep, ref_g = oracle.select_full(wl.as_f64(X), TAU)
    tol = 2e-3 if dtype == "bf16" else 1e-5
    assert np.max(np.abs(gamma.cpu().numpy()[0] - ref_g)) <= tol
    assert lists(idx, cnt)[0].tolist() == ref_rep.tolist()
    out = ada.ada_cascade_step(ctx, Xv, TAU, idx, cnt)
    ref = oracle.cascade_step(wl.as_f64(X), TAU, ref_rep)
    assert lists(out.rep_out, out.rep_out_cnt)[0].tolist() == ref.rep.tolist()
    assert np.max(np.abs(out.gamma_cross.cpu().numpy()[0] - ref.gamma_cross)) <= tol
    near, _ = ada.ada_nearest_rep(ctx, Xv, out.rep_out, out.rep_out_cnt)
    assert near.cpu().numpy()[0].tolist() == oracle.nearest(wl.as_f64(X), ref.rep)[0].tolist()
    assert ada.ada_device_status(ctx)[0] == 0
    ada.ada_destroy(ctx)


def test_bounded_wait_runs_out_and_the_context_survives(ada):
    """The in-kernel waits have a limit: a wait on a flag nothing sets ends with a status the
    host can read (no trap, no hang), and the context keeps working afterwards."""
    from parity import check_full
    ctx = ada.ada_create(1, 256, 64, ada.ADA_BF16)
    ada.ada_selftest_wait_timeout(ctx, limit_ms=50)
    st, _ = ada.ada_device_status(ctx)
    assert st == 7 and ada.status_string(st) == "ADA_ERR_TIMEOUT"
    assert ada.ada_device_status(ctx)[0] == 0                   # reading clears it
    band, reps = check_full(ctx, clustered(256, 64, 3, "bf16"), TAU)
    assert len(reps[0]) > 0
    ada.ada_destroy(ctx)


def test_host_entry_points_match_device_ones(ada):
    from parity import lists, to_device
    cfg = wl.scaled(wl.CONFIGS[2], B=3, T=700, d=256, L=2)
    Xs, _ = wl.generate_all(cfg)
    ctx = ada.ada_create(3, 700, 256, ada.ADA_BF16)
    d0, d1 = to_device(Xs[0]), to_device(Xs[1])
    ri, rc, g = ada.ada_select_full(ctx, d0, cfg.tau)
    out = ada.ada_cascade_step(ctx, d1, cfg.tau, ri, rc)
    h0, h1 = d0.cpu().pin_memory(), d1.cpu().pin_memory()
    i32 = lambda *s: torch.empty(s, dtype=torch.int32).pin_memory()
    hri, hrc, hg = i32(3, 700), i32(3), torch.empty(3, 700).pin_memory()
    ada.ada_select_full_host(ctx, h0, cfg.tau, hri, hrc, hg)
    assert [a.tolist() for a in lists(hri, hrc)] == [a.tolist() for a in lists(ri, rc)]
    assert torch.equal(hg, g.cpu())
    ro, roc, ai, ac, mi, mc = i32(3, 700), i32(3), i32(3, 700), i32(3), i32(3, 700), i32(3)
    ada.ada_cascade_step_host(ctx, h1, cfg.tau, hri, hrc, ro, roc, ai, ac, mi, mc)
    assert [a.tolist() for a in lists(ro, roc)] == [a.tolist() for a in lists(out.rep_out, out.rep_out_cnt)]
    assert [a.tolist() for a in lists(ai, ac)] == [a.tolist() for a in lists(out.add_idx, out.add_cnt)]
    assert [a.tolist() for a in lists(mi, mc)] == [a.tolist() for a in lists(out.rem_idx, out.rem_cnt)]
    ada.ada_destroy(ctx)


def test_repeated_runs_are_bit_identical(ada):
    from parity import to_device
    cfg = wl.scaled(wl.CONFIGS[3], T=1024, d=512, L=1, P=100)
    Xd = to_device(next(wl.generate_layers(cfg)).X)
    ctx = ada.ada_create(1, 1024, 512, ada.ADA_BF16)
    a = ada.ada_select_full(ctx, Xd, cfg.tau)
    b = ada.ada_select_full(ctx, Xd, cfg.tau)
    assert torch.equal(a[2], b[2]) and torch.equal(a[1], b[1])
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("cfg_id", [1, 2])
def test_dependent_launch_on_and_off_give_identical_results(ada, cfg_id):
    """The launch attribute changes when a kernel's blocks may be placed, never what it computes:
    a chain of calls with programmatic dependent launch on (default) and off, bit for bit."""
    from parity import to_device
    cfg = wl.scaled(wl.CONFIGS[cfg_id], L=4)
    layers = [to_device(lb.X) for lb in wl.generate_layers(cfg, seed=1)]
    res = []
    for on in (True, False):
        ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_F32 if cfg.dtype == "f32" else ada.ADA_BF16)
        ada.ada_set_dependent_launch(ctx, on)
        idx, cnt, g = ada.ada_select_full(ctx, layers[0], cfg.tau)
        out = [cnt.clone(), g.clone()] + [idx[b, :int(cnt[b])].clone() for b in range(cfg.B)]
        for X in layers[1:]:
            o = ada.ada_cascade_step(ctx, X, cfg.tau, idx, cnt)
            idx, cnt = o.rep_out, o.rep_out_cnt
            out += [o.rep_out_cnt.clone(), o.add_cnt.clone(), o.rem_cnt.clone(), o.gamma_rep.clone(),
                    o.gamma_cross.clone()]
            for b in range(cfg.B):
                out.append(o.rep_out[b, :int(o.rep_out_cnt[b])].clone())
        st, _ = ada.ada_device_status(ctx)
        assert st == 0
        res.append(out)
        ada.ada_destroy(ctx)
    assert len(res[0]) == len(res[1])
    for a, b in zip(*res):
        assert torch.equal(a, b)


@pytest.mark.parametrize("T,d", [(130, 72), (257, 768), (600, 8), (1500, 256)])
def test_row_compaction_of_the_cross_step_small_shapes(ada, T, d):
    """Algorithm 1 line 6 over the copied-out rows (pair kernel, forced on at any length):
    inherited sets of two fifths of the tokens and more, literal and causal, against the oracle."""
    from parity import check_cascade
    ctx = ada.ada_create(1, T, d, ada.ADA_BF16)
    ada.ada_set_engine(ctx, ada.ADA_ENGINE_TCGEN05_PAIR)
    ada.ada_set_row_compaction(ctx, 1)
    X = clustered(T, d, 4000 + T + d, "bf16")
    rng = np.random.default_rng(T + d)
    sets = [list(range(T)), list(range(0, T, 2)), list(range(1, T, 2)), list(range(T // 2, T)),
            list(range(0, T // 2 + 1)), sorted(rng.choice(T, (T * 3) // 5, replace=False).tolist()),
            list(range(0, T, 3))]                      # the last one is below the threshold: streamed
    for R in sets:
        for causal in (False, True):
            check_cascade(ctx, X, TAU, [R], causal=causal)
    ada.ada_destroy(ctx)


def test_row_compaction_batched_and_on_and_off_agree(ada):
    """Several sequences with different large sets in one call; the lists and gammas with the
    row compaction on and off are identical bit for bit (it changes which rows are loaded, not
    what is computed for them)."""
    from parity import check_cascade, to_device
    cfg = wl.scaled(wl.CONFIGS[2], B=3, T=700, d=264, L=2)
    Xs, _ = wl.generate_all(cfg)
    rng = np.random.default_rng(9)
    Rs = [sorted(rng.choice(cfg.T, n, replace=False).tolist()) for n in (300, 699, 420)]
    outs = []
    for min_rows in (1, 1 << 30):
        ctx = ada.ada_create(3, cfg.T, cfg.d, ada.ADA_BF16)
        ada.ada_set_engine(ctx, ada.ADA_ENGINE_TCGEN05_PAIR)
        ada.ada_set_row_compaction(ctx, min_rows)
        check_cascade(ctx, Xs[1], cfg.tau, Rs)
        rin = np.zeros((3, cfg.T), dtype=np.int32)
        for b, r in enumerate(Rs):
            rin[b, :len(r)] = r
        o = ada.ada_cascade_step(ctx, to_device(Xs[1]), cfg.tau, torch.from_numpy(rin).cuda(),
                                 torch.tensor([len(r) for r in Rs], dtype=torch.int32).cuda())
        outs.append([o.rep_out.clone(), o.rep_out_cnt.clone(), o.add_cnt.clone(), o.rem_cnt.clone(),
                     o.gamma_rep.clone(), o.gamma_cross.clone()])
        assert ada.ada_device_status(ctx)[0] == 0
        ada.ada_destroy(ctx)
    for a, b in zip(*outs[:2]):
        if a.dtype == torch.int32 and a.dim() == 2:      # list capacity beyond the counts is unspecified
            for s in range(3):
                n = int(outs[0][1][s])
                assert torch.equal(a[s, :n], b[s, :n])
        else:
            assert torch.equal(a, b)


def test_rejected_list_on_the_pair_kernel_with_row_compaction(ada):
    """A list that is not ascending is reported and leaves everything in bounds, also where the
    launch copies the rows outside the set (their positions then make no sense); the context
    works afterwards."""
    from parity import check_cascade
    T, d = 192, 64
    ctx = ada.ada_create(1, T, d, ada.ADA_BF16)
    ada.ada_set_engine(ctx, ada.ADA_ENGINE_TCGEN05_PAIR)
    ada.ada_set_row_compaction(ctx, 1)
    X = clustered(T, d, 77, "bf16")
    Xd = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).cuda()
    bad = torch.zeros((1, T), dtype=torch.int32)
    bad[0, :120] = torch.arange(150, 30, -1, dtype=torch.int32)      # descending
    ada.ada_cascade_step(ctx, Xd, TAU, bad.cuda(), torch.tensor([120], dtype=torch.int32).cuda())
    assert ada.ada_device_status(ctx)[0] == 5
    bad[0, :120] = torch.arange(0, 120, dtype=torch.int32)
    bad[0, 60] = 5000                                                 # out of range
    ada.ada_cascade_step(ctx, Xd, TAU, bad.cuda(), torch.tensor([120], dtype=torch.int32).cuda())
    assert ada.ada_device_status(ctx)[0] == 5
    check_cascade(ctx, X, TAU, [list(range(0, T, 2))])
    ada.ada_destroy(ctx)
