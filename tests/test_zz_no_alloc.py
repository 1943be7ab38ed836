"""The allocation-free entry point against the context-based one (collected last on purpose).

Some users of the library may not allocate device memory at call time -- all of HBM
belongs to their own pool, or an allocation's device-wide synchronisation is not
acceptable, or their host application forbids it -- so they cannot create a context.
ada_select_full_noalloc serves them from a fixed scratch array inside the library.  This
test calls it through the C ABI twice in a row (the scratch is shared between calls and
keeps old contents, so the second call checks that stale state does no harm) and compares
with ada_select_full on the same inputs, and with the fp64 oracle (gamma within the path's
tolerance, the set equal outside the tolerance band around the threshold).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_03110_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _layer(cfg, seed):
    """(host array of one sequence, the same on the device in its storage type)"""
    X = next(wl.generate_layers(cfg, seed=seed)).X
    if X.dtype == np.uint16:
        return X[0], torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).cuda()
    return X[0], torch.from_numpy(X).cuda()


@pytest.mark.parametrize("base,T,d", [(3, 1500, 512), (1, 512, 768)])
def test_noalloc_matches_context_entry_point_twice(base, T, d):
    from paper_2605_03110_b200 import binding as ada
    cfg = wl.scaled(wl.CONFIGS[base], T=T, d=d, L=1, P=max(8, T // 12))
    tol = 2e-3 if cfg.dtype == "bf16" else 1e-5
    ctx = ada.ada_create(1, T, d, ada.ADA_BF16 if cfg.dtype == "bf16" else ada.ADA_F32)
    if cfg.dtype == "f32":
        # fp32 storage runs on the FFMA kernel in the allocation-free call: compare like with like
        ada.ada_set_engine(ctx, ada.ADA_ENGINE_FFMA)
    idx = torch.empty(T, dtype=torch.int32, device="cuda")
    cnt = torch.empty(1, dtype=torch.int32, device="cuda")
    gam = torch.empty(T, dtype=torch.float32, device="cuda")
    for call, seed in enumerate((0, 1)):          # two calls in a row, different inputs
        Xh, X = _layer(cfg, seed)
        ref_idx, ref_cnt, ref_gamma = ada.ada_select_full(ctx, X, cfg.tau)
        idx.fill_(-1)
        ada.ada_select_full_noalloc(X, cfg.tau, idx, cnt, gam)
        torch.cuda.synchronize()
        r = int(cnt[0])
        assert r == int(ref_cnt[0]) and 0 < r < T, f"call {call}"
        assert torch.equal(idx[:r], ref_idx[0, :r]), f"call {call}"
        assert float((gam - ref_gamma[0]).abs().max()) <= tol, f"call {call}"
        # and against the oracle
        from parity import check_set
        o_rep, o_gamma = oracle.select_full(wl.as_f64(Xh), cfg.tau)
        assert np.max(np.abs(gam.cpu().numpy() - o_gamma)) <= tol, f"call {call}"
        got = idx[:r].cpu().numpy()
        if check_set(got, o_gamma, np.arange(T), 1.0 - cfg.tau * cfg.tau, tol) == 0:
            assert got.tolist() == o_rep.tolist(), f"call {call}"
    ada.ada_destroy(ctx)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2605_03110_b200 import binding as ada
    T = ada.ADA_NOALLOC_MAX_T + 8
    X = torch.zeros(T, 8, dtype=torch.bfloat16, device="cuda")
    idx = torch.empty(T, dtype=torch.int32, device="cuda")
    cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    with pytest.raises(ada.AdaError) as e:
        ada.ada_select_full_noalloc(X, 0.3, idx, cnt)
    assert e.value.status == 3 and "ADA_NOALLOC_MAX_T" in str(e.value)
    torch.cuda.synchronize()
    assert int(cnt[0]) == -7                      # nothing was enqueued
