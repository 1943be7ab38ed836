"""Shared helpers of the GPU parity tests: device upload, band-aware set comparison."""
import numpy as np
import torch

import oracle
from paper_2605_03110_b200 import binding as ada
from paper_2605_03110_b200 import workloads as wl

TOL = {"f32": 1e-5, "bf16": 2e-3}      # |gamma_gpu - gamma_oracle| allowed (absolute)


def to_device(X: np.ndarray) -> torch.Tensor:
    """(B,T,d) float32 or uint16 (bf16 bits) -> cuda tensor of the storage type."""
    if X.dtype == np.uint16:
        return torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).cuda()
    return torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).cuda()


def dtype_name(X: np.ndarray) -> str:
    return "bf16" if X.dtype == np.uint16 else "f32"


def lists(idx: torch.Tensor, cnt: torch.Tensor):
    idx, cnt = idx.cpu().numpy(), cnt.cpu().numpy()
    return [idx[b, :cnt[b]].copy() for b in range(idx.shape[0])]


def check_set(got, gamma_ref, candidates, thr, tol):
    """got: selected subset of `candidates`; the reference selects gamma_ref < thr.
    Returns the number of tolerated band disagreements; asserts on any other."""
    got = set(int(x) for x in got)
    assert got <= set(int(c) for c in candidates)
    band = 0
    for t in candidates:
        ref_in = gamma_ref[t] < thr
        if (int(t) in got) != ref_in:
            assert abs(gamma_ref[t] - thr) <= tol, (int(t), gamma_ref[t])
            band += 1
    return band


def check_full(ctx, Xnp, tau, stream=None, heads=False):
    """ada_select_full vs the oracle on every sequence.  Returns band count.
    heads: Xnp is (T, h, d_h); the device gets it as it is (ada_select_full_heads), the oracle
    gets each head as a sequence of its own."""
    tol = TOL[dtype_name(Xnp)]
    thr = 1.0 - tau * tau
    Xd = to_device(Xnp)
    if heads:
        rep_idx, rep_cnt, gamma = ada.ada_select_full_heads(ctx, Xd, tau)
        Xnp = np.ascontiguousarray(Xnp.transpose(1, 0, 2))
    else:
        rep_idx, rep_cnt, gamma = ada.ada_select_full(ctx, Xd, tau)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0, ada.status_string(st)
    reps = lists(rep_idx, rep_cnt)
    g = gamma.cpu().numpy()
    band = 0
    for b in range(Xnp.shape[0]):
        ref_rep, ref_g = oracle.select_full(wl.as_f64(Xnp[b]), tau)
        assert np.max(np.abs(g[b] - ref_g), initial=0.0) <= tol
        assert np.all(np.diff(reps[b]) > 0)
        nb = check_set(reps[b], ref_g, np.arange(Xnp.shape[1]), thr, tol)
        if nb == 0:
            assert reps[b].tolist() == ref_rep.tolist()
        band += nb
    return band, reps


def check_cascade(ctx, Xnp, tau, rep_in_lists, causal=False, heads=False):
    """ada_cascade_step vs the oracle, same inherited sets on both sides (heads: as check_full)."""
    tol = TOL[dtype_name(Xnp)]
    thr = 1.0 - tau * tau
    Xd = to_device(Xnp)
    if heads:
        Xnp = np.ascontiguousarray(Xnp.transpose(1, 0, 2))
    B, T, _ = Xnp.shape
    rin = np.zeros((B, T), dtype=np.int32)
    rcnt = np.zeros(B, dtype=np.int32)
    for b, r in enumerate(rep_in_lists):
        rin[b, :len(r)] = r
        rcnt[b] = len(r)
    step = ada.ada_cascade_step_heads if heads else ada.ada_cascade_step
    out = step(ctx, Xd, tau, torch.from_numpy(rin).cuda(), torch.from_numpy(rcnt).cuda(),
               flags=ada.ADA_CROSS_CAUSAL if causal else 0)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0, ada.status_string(st)
    rep, add, rem = lists(out.rep_out, out.rep_out_cnt), lists(out.add_idx, out.add_cnt), \
        lists(out.rem_idx, out.rem_cnt)
    g_rep, g_cross = out.gamma_rep.cpu().numpy(), out.gamma_cross.cpu().numpy()
    band = 0
    refs = []
    for b in range(B):
        X64 = wl.as_f64(Xnp[b])
        R = np.asarray(rep_in_lists[b], dtype=np.int32)
        ref = oracle.cascade_step(X64, tau, R, causal=causal)
        # lines 3-5
        g_rep_tok = np.zeros(T)
        g_rep_tok[R] = ref.gamma_rep
        assert np.max(np.abs(g_rep[b] - g_rep_tok), initial=0.0) <= tol
        kept = np.setdiff1d(R, rem[b])
        nb = check_set(kept, g_rep_tok, R, thr, tol)
        if nb:   # continue from the GPU's valid set (differs only inside the band)
            ref = oracle.cascade_step(X64, tau, R, causal=causal,
                                      force_valid=np.isin(R, kept).astype(np.uint8))
        else:
            assert rem[b].tolist() == ref.rem.tolist()
        # lines 6-9
        nonrep = np.setdiff1d(np.arange(T), R)
        assert np.max(np.abs(g_cross[b] - ref.gamma_cross), initial=0.0) <= tol
        na = check_set(add[b], ref.gamma_cross, nonrep, thr, tol)
        if na == 0:
            assert add[b].tolist() == ref.add.tolist()
        if nb == 0 and na == 0:
            assert rep[b].tolist() == ref.rep.tolist()
        # lines 10-11 and list structure
        assert rep[b].tolist() == sorted(set(kept.tolist()) | set(add[b].tolist()))
        assert np.all(np.diff(rep[b]) > 0) and np.all(np.diff(add[b]) > 0) and np.all(np.diff(rem[b]) > 0)
        assert len(rep[b]) == len(R) + len(add[b]) - len(rem[b])
        band += nb + na
        refs.append(ref)
    return band, rep, refs
