"""Cascade steps with a device-resident threshold that follows the turnover (Section 8.1),
through the C ABI against the oracle (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ada():
    from paper_2605_03110_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return binding


def run_chain(ada, cfg, tau0, policy, causal=False, seed=0, engine=0):
    """Free-running GPU chain with per-sequence thresholds; every step is checked against the
    oracle run with the same threshold and the same inherited set, the threshold state against
    the oracle's update rule fed with the step's own counts (bit for bit)."""
    from parity import TOL, check_set, lists, to_device
    tol = TOL[cfg.dtype]
    B, T = cfg.B, cfg.T
    ctx = ada.ada_create(B, T, cfg.d, ada.ADA_F32 if cfg.dtype == "f32" else ada.ADA_BF16)
    ada.ada_set_engine(ctx, engine)
    tau = np.array(tau0, dtype=np.float64)
    tau_dev = torch.from_numpy(tau.copy()).cuda()
    turn = torch.empty(B, dtype=torch.float32, device="cuda")
    pol = None if policy is None else ada.TauPolicy(*policy)
    R, idx, cnt = None, None, None
    band_total, history = 0, [tau.copy()]
    for lb in wl.generate_layers(cfg, seed=seed):
        Xd = to_device(lb.X)
        if lb.layer == 0:
            # layer 0: Definition 1 with each sequence's own threshold (one call per sequence)
            idx = torch.zeros((B, T), dtype=torch.int32, device="cuda")
            cnt = torch.zeros(B, dtype=torch.int32, device="cuda")
            for b in range(B):
                i1, c1, _ = ada.ada_select_full(ctx, Xd[b:b + 1], float(tau[b]))
                idx[b], cnt[b] = i1[0], c1[0]
            R = lists(idx, cnt)
            for b in range(B):
                assert R[b].tolist() == oracle.select_full(wl.as_f64(lb.X[b]), float(tau[b]))[0].tolist()
            continue
        out = ada.ada_cascade_step_adaptive(ctx, Xd, tau_dev, pol, idx, cnt, turnover=turn,
                                            flags=ada.ADA_CROSS_CAUSAL if causal else 0)
        st, _ = ada.ada_device_status(ctx)
        assert st == 0, ada.status_string(st)
        rep, add, rem = lists(out.rep_out, out.rep_out_cnt), lists(out.add_idx, out.add_cnt), \
            lists(out.rem_idx, out.rem_cnt)
        g_rep, g_cross = out.gamma_rep.cpu().numpy(), out.gamma_cross.cpu().numpy()
        tau_new = tau_dev.cpu().numpy()
        rho_dev = turn.cpu().numpy()
        for b in range(B):
            thr = 1.0 - tau[b] * tau[b]
            ref = oracle.cascade_step(wl.as_f64(lb.X[b]), float(tau[b]), R[b], causal=causal)
            g_rep_tok = np.zeros(T)
            g_rep_tok[R[b]] = ref.gamma_rep
            assert np.max(np.abs(g_rep[b] - g_rep_tok), initial=0.0) <= tol
            kept = np.setdiff1d(R[b], rem[b])
            nb = check_set(kept, g_rep_tok, R[b], thr, tol)
            if nb:
                ref = oracle.cascade_step(wl.as_f64(lb.X[b]), float(tau[b]), R[b], causal=causal,
                                          force_valid=np.isin(R[b], kept).astype(np.uint8))
            assert np.max(np.abs(g_cross[b] - ref.gamma_cross), initial=0.0) <= tol
            na = check_set(add[b], ref.gamma_cross, np.setdiff1d(np.arange(T), R[b]), thr, tol)
            if nb == 0 and na == 0:
                assert rep[b].tolist() == ref.rep.tolist()
                assert add[b].tolist() == ref.add.tolist() and rem[b].tolist() == ref.rem.tolist()
            band_total += nb + na
            # Eq. 6 and the update rule, from this step's own counts
            rho = oracle.turnover(len(add[b]), len(rem[b]), len(R[b]))
            if np.isnan(rho):
                assert np.isnan(rho_dev[b])
            else:
                assert rho_dev[b] == np.float32(rho)
            want = tau[b] if policy is None else oracle.tau_update(tau[b], rho, *policy)
            assert tau_new[b] == want, (b, lb.layer, tau_new[b], want)
        tau = tau_new.copy()
        history.append(tau.copy())
        R, idx, cnt = rep, out.rep_out, out.rep_out_cnt
    ada.ada_destroy(ctx)
    return band_total, np.array(history)


@pytest.mark.parametrize("causal", [False, True])
def test_adaptive_chain_bf16_batched(ada, causal):
    cfg = wl.scaled(wl.CONFIGS[2], B=3, T=700, d=256, L=7, P=60)
    band, hist = run_chain(ada, cfg, [0.3, 0.2, 0.45], (0.08, 0.5, 0.1, 0.6), causal=causal)
    assert band == 0
    assert np.all(hist >= 0.1) and np.all(hist <= 0.6)
    assert not np.array_equal(hist[0], hist[-1])          # the thresholds did move


# engines: 0 automatic, 1 FFMA kernel, 3 pair-CTA tensor-core kernel (each reads the per-sequence
# threshold in its own epilogue)
@pytest.mark.parametrize("engine", [0, 1, 3])
def test_adaptive_chain_fp32(ada, engine):
    cfg = wl.scaled(wl.CONFIGS[1], T=500, d=192, L=6, P=50)
    band, hist = run_chain(ada, cfg, [0.3], (0.05, 1.0, 0.15, 0.5), engine=engine)
    assert band == 0


@pytest.mark.parametrize("engine", [1, 2, 3])
def test_adaptive_chain_bf16_on_every_engine(ada, engine):
    cfg = wl.scaled(wl.CONFIGS[2], B=2, T=520, d=320, L=5, P=50)
    band, hist = run_chain(ada, cfg, [0.25, 0.4], (0.08, 0.5, 0.1, 0.6), engine=engine)
    assert band == 0


def test_strong_gain_runs_into_the_bounds(ada):
    cfg = wl.scaled(wl.CONFIGS[2], B=2, T=400, d=128, L=6, P=40)
    _, hist = run_chain(ada, cfg, [0.3, 0.3], (0.0, 50.0, 0.2, 0.4))
    # target 0 and a large gain: any turnover at all drives tau to its lower bound, where it stays
    assert np.all(hist[-1] == 0.2)
    assert np.all(np.diff(hist, axis=0) <= 0) and set(np.unique(hist)) <= {0.2, 0.3}


def test_no_policy_equals_the_fixed_threshold_step_bit_for_bit(ada):
    from parity import to_device
    cfg = wl.scaled(wl.CONFIGS[2], B=4, T=900, d=384, L=3, P=80)
    layers = [to_device(lb.X) for lb in wl.generate_layers(cfg, seed=2)]
    ctx = ada.ada_create(cfg.B, cfg.T, cfg.d, ada.ADA_BF16)
    idx, cnt, _ = ada.ada_select_full(ctx, layers[0], cfg.tau)
    tau_dev = torch.full((cfg.B,), cfg.tau, dtype=torch.float64, device="cuda")
    a = ada.ada_cascade_step(ctx, layers[1], cfg.tau, idx, cnt)
    b = ada.ada_cascade_step_adaptive(ctx, layers[1], tau_dev, None, idx, cnt)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    assert torch.equal(tau_dev.cpu(), torch.full((cfg.B,), cfg.tau, dtype=torch.float64))
    for name in ("rep_out_cnt", "add_cnt", "rem_cnt", "gamma_rep", "gamma_cross"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    for s in range(cfg.B):
        n = int(a.rep_out_cnt[s])
        assert torch.equal(a.rep_out[s, :n], b.rep_out[s, :n])
    ada.ada_destroy(ctx)


def test_empty_inherited_set_and_error_paths(ada):
    ctx = ada.ada_create(2, 64, 64, ada.ADA_BF16)
    X = torch.randn(2, 64, 64, device="cuda").to(torch.bfloat16)
    idx = torch.zeros((2, 64), dtype=torch.int32, device="cuda")
    cnt = torch.tensor([0, 1], dtype=torch.int32, device="cuda")   # empty set / token 0 only
    tau_dev = torch.tensor([0.3, 0.3], dtype=torch.float64, device="cuda")
    turn = torch.zeros(2, dtype=torch.float32, device="cuda")
    pol = ada.TauPolicy(0.1, 0.5, 0.1, 0.6)
    out = ada.ada_cascade_step_adaptive(ctx, X, tau_dev, pol, idx, cnt, turnover=turn)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    t = turn.cpu().numpy()
    assert np.isnan(t[0]) and int(out.add_cnt[0]) == 64       # Eq. 6 undefined: tau stays
    assert tau_dev[0].item() == 0.3
    rho1 = (int(out.add_cnt[1]) + int(out.rem_cnt[1])) / 1.0
    assert t[1] == np.float32(rho1)
    assert tau_dev[1].item() == oracle.tau_update(0.3, rho1, 0.1, 0.5, 0.1, 0.6)
    # host-checked faults
    for bad in (ada.TauPolicy(0.1, -1.0, 0.1, 0.6), ada.TauPolicy(0.1, 0.5, 0.0, 0.6),
                ada.TauPolicy(0.1, 0.5, 0.5, 0.4), ada.TauPolicy(0.1, 0.5, 0.1, 1.0),
                ada.TauPolicy(float("nan"), 0.5, 0.1, 0.6)):
        with pytest.raises(ada.AdaError) as e:
            ada.ada_cascade_step_adaptive(ctx, X, tau_dev, bad, idx, cnt)
        assert e.value.status == 1
    # device-checked fault: a threshold state outside (0, 1); the context stays usable
    bad_tau = torch.tensor([0.3, 1.5], dtype=torch.float64, device="cuda")
    ada.ada_cascade_step_adaptive(ctx, X, bad_tau, None, idx, cnt)
    st, _ = ada.ada_device_status(ctx)
    assert st == 8 and ada.status_string(st) == "ADA_ERR_BAD_TAU"
    ada.ada_cascade_step_adaptive(ctx, X, tau_dev, None, idx, cnt)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0
    ada.ada_destroy(ctx)
