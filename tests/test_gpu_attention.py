"""Attention on the representative set (Section 2.3, Eq. 2) on the GPU against the oracle.

Tolerance: the (unnormalised) probabilities are rounded to bf16 between the two contractions
(relative error 2^-9 each) while their row sum is taken in fp32 from the unrounded values, so an
output element is off by at most about 2^-9 max|V|.  The tests allow 2^-8 max|V|.
"""
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


def bf16_round(a):
    return wl.bf16_bits_to_f32(wl.f32_to_bf16_bits(a.astype(np.float32)))


def dev_bf16(a):
    return torch.from_numpy(wl.f32_to_bf16_bits(a).view(np.int16)).view(torch.bfloat16).cuda()


def run_case(ada, ctx, Q, K, V, R, near, causal):
    T, h, d_h = Q.shape
    idx = torch.zeros(T, dtype=torch.int32)
    idx[:len(R)] = torch.tensor(R, dtype=torch.int32)
    cnt = torch.tensor([len(R)], dtype=torch.int32)
    near_d = None if near is None else torch.from_numpy(np.asarray(near, dtype=np.int32)).cuda()
    out = ada.ada_attention_reps(ctx, dev_bf16(Q), dev_bf16(K), dev_bf16(V), idx.cuda(), cnt.cuda(),
                                 nearest_idx=near_d, flags=ada.ADA_ATTN_CAUSAL if causal else 0)
    st, _ = ada.ada_device_status(ctx)
    assert st == 0, ada.status_string(st)
    ref = oracle.attention_reps(Q.astype(np.float64), K.astype(np.float64), V.astype(np.float64), R,
                                nearest_idx=near, causal=causal)
    tol = 2.0 ** -8 * max(1e-30, float(np.max(np.abs(V))))
    got = out.cpu().numpy()
    assert np.max(np.abs(got - ref)) <= tol, float(np.max(np.abs(got - ref)))
    return got


@pytest.mark.parametrize("T,h,d_h", [(1, 1, 16), (5, 3, 64), (130, 2, 128), (300, 3, 80), (700, 1, 32)])
@pytest.mark.parametrize("causal", [False, True])
def test_small_shapes(ada, T, h, d_h, causal):
    rng = np.random.default_rng(T * 31 + h * 7 + d_h)
    Q, K, V = (bf16_round(rng.standard_normal((T, h, d_h))) for _ in range(3))
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    sets = [list(range(T)), [0], [T - 1], list(range(0, T, 3)),
            sorted(rng.choice(T, max(1, T // 2), replace=False).tolist())]
    for R in sets:
        near = np.asarray([R[int(rng.integers(len(R)))] for _ in range(T)], dtype=np.int32)
        near[R] = R
        run_case(ada, ctx, Q, K, V, R, near, causal)
        run_case(ada, ctx, Q, K, V, R, None, causal)     # representatives' rows only
    ada.ada_destroy(ctx)


def test_empty_set_gives_zero_rows(ada):
    rng = np.random.default_rng(3)
    T, h, d_h = 40, 2, 16
    Q, K, V = (bf16_round(rng.standard_normal((T, h, d_h))) for _ in range(3))
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    got = run_case(ada, ctx, Q, K, V, [], np.full(T, -1, dtype=np.int32), False)
    assert np.all(got == 0.0)
    ada.ada_destroy(ctx)


def test_constant_values_pass_through(ada):
    """Softmax rows sum to one: with V = 1 every written row is 1 up to the rounding of P."""
    rng = np.random.default_rng(4)
    T, h, d_h = 500, 2, 64
    Q, K = (bf16_round(rng.standard_normal((T, h, d_h))) for _ in range(2))
    V = np.ones((T, h, d_h), dtype=np.float32)
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    R = list(range(0, T, 2))
    got = run_case(ada, ctx, Q, K, V, R, None, False)
    assert np.max(np.abs(got[R] - 1.0)) <= 2.0 ** -8
    ada.ada_destroy(ctx)


def test_many_key_tiles_random(ada):
    """r = 1400 of T = 2048: eleven key tiles per query tile (six for one warp set, five for the other)."""
    rng = np.random.default_rng(5)
    T, h, d_h = 2048, 4, 128
    Q, K, V = (bf16_round(rng.standard_normal((T, h, d_h))) for _ in range(3))
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    R = sorted(rng.choice(T, 1400, replace=False).tolist())
    for causal in (False, True):
        run_case(ada, ctx, Q, K, V, R, None, causal)
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("causal", [False, True])
def test_more_work_items_than_sms(ada, causal):
    """The CTAs are persistent: with 20 query tiles x 16 heads = 320 work items every CTA takes two
    or three in a row, its rings, barriers and accumulators carried over (under the causal mask
    with a different number of key tiles each time).  A second set with 7 query tiles leaves most
    CTAs one item and some none."""
    rng = np.random.default_rng(11 + causal)
    T, h, d_h = 2560, 16, 32
    Q, K, V = (bf16_round(rng.standard_normal((T, h, d_h))) for _ in range(3))
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    near = np.arange(T, dtype=np.int32)
    run_case(ada, ctx, Q, K, V, list(range(T)), near, causal)
    R = sorted(rng.choice(T, 800, replace=False).tolist())
    run_case(ada, ctx, Q, K, V, R, None, causal)
    ada.ada_destroy(ctx)


@pytest.mark.parametrize("growth", [0.5, 1.0, 1.6, 4.0])
@pytest.mark.parametrize("causal", [False, True])
def test_row_maximum_that_moves_across_key_tiles(ada, growth, causal):
    """The kernel walks the key tiles once and rescales its accumulator only when a row's
    maximum has moved far: keys whose scale grows from one 128-key tile to the next make the
    maximum move a little (1.6: some rows rescale on some tiles), a lot (4: every row on every
    tile) or never (1, 0.5: the first tile holds it), and the result must not depend on it."""
    rng = np.random.default_rng(int(growth * 10) + causal)
    T, h, d_h = 900, 2, 64
    Q, K, V = (rng.standard_normal((T, h, d_h)) for _ in range(3))
    K *= (growth ** (np.arange(T) // 128))[:, None, None]
    K[5:9] *= 6.0                                  # and a few early keys that dominate some rows
    Q, K, V = bf16_round(Q), bf16_round(K), bf16_round(V)
    ctx = ada.ada_create(1, T, h * d_h, ada.ADA_BF16)
    for R in (list(range(T)), list(range(3, T, 2))):
        run_case(ada, ctx, Q, K, V, R, None, causal)
    ada.ada_destroy(ctx)


def test_selection_to_attention_pipeline_on_config3(ada):
    """The hand-off the paper describes: selection -> nearest-representative map -> attention on
    the representatives, expanded to all tokens; the layer's activations stand in for Q, K, V
    (32 heads of 128), the whole chain on the device, compared with the oracle's chain."""
    from parity import lists, to_device
    cfg = wl.CONFIGS[3]
    lb = next(wl.generate_layers(cfg, seed=0, n_layers=1))
    Xd = to_device(lb.X)                                   # (1, T, d) bf16
    T, h, d_h = cfg.T, 32, cfg.d // 32
    ctx = ada.ada_create(1, T, cfg.d, ada.ADA_BF16)
    idx, cnt, _ = ada.ada_select_full(ctx, Xd, cfg.tau)
    near, _ = ada.ada_nearest_rep(ctx, Xd, idx, cnt)
    X3 = Xd[0].view(T, h, d_h)
    out = ada.ada_attention_reps(ctx, X3, X3, X3, idx[0], cnt, nearest_idx=near[0])
    assert ada.ada_device_status(ctx)[0] == 0
    X64 = wl.as_f64(lb.X[0])
    R, _ = oracle.select_full(X64, cfg.tau)
    assert lists(idx, cnt)[0].tolist() == R.tolist()
    near_ref, _ = oracle.nearest(X64, R)
    near_gpu = near[0].cpu().numpy()
    Xh = X64.reshape(T, h, d_h)
    ref = oracle.attention_reps(Xh, Xh, Xh, R, nearest_idx=near_gpu)   # same map on both sides
    tol = 2.0 ** -8 * float(np.max(np.abs(X64)))
    assert np.max(np.abs(out.cpu().numpy() - ref)) <= tol
    # the map itself agrees with the oracle's wherever the maximum is unique (checked elsewhere
    # with the tolerance rule); here: every token's nearest representative is a representative
    assert set(near_gpu.tolist()) <= set(R.tolist())
    assert np.mean(near_gpu == near_ref) > 0.999
    ada.ada_destroy(ctx)


def test_error_paths(ada):
    ctx = ada.ada_create(1, 64, 64, ada.ADA_BF16)
    q = torch.zeros(64, 1, 64, dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros(64, dtype=torch.int32, device="cuda")
    cnt = torch.ones(1, dtype=torch.int32, device="cuda")
    with pytest.raises(ada.AdaError) as e:                      # head width not a multiple of 16
        x = torch.zeros(64, 1, 24, dtype=torch.bfloat16, device="cuda")
        ada.ada_attention_reps(ctx, x, x, x, idx, cnt)
    assert e.value.status == 2
    with pytest.raises(ada.AdaError) as e:                      # unknown flag
        ada.ada_attention_reps(ctx, q, q, q, idx, cnt, flags=2)
    assert e.value.status == 1
    with pytest.raises(ada.AdaError) as e:                      # above the context's width
        x = torch.zeros(64, 2, 64, dtype=torch.bfloat16, device="cuda")
        ada.ada_attention_reps(ctx, x, x, x, idx, cnt)
    assert e.value.status == 3
    with pytest.raises(TypeError):
        ada.ada_attention_reps(ctx, q.half(), q.half(), q.half(), idx, cnt)
    ada.ada_destroy(ctx)


def test_two_stream_pipeline_matches_the_serial_order(ada):
    """Section 8.4: selection of layer l+1 on one stream while layer l's nearest-representative map
    and attention run on another; the results are those of the serial order, bit for bit."""
    from paper_2605_03110_b200.pipeline import SelectionAttentionPipeline
    cfg = wl.scaled(wl.CONFIGS[3], T=1024, d=1024, L=5, P=100, rho=0.05)
    dev = torch.device("cuda", 0)
    T, h, d_h = cfg.T, 8, cfg.d // 8
    layers = [torch.from_numpy(lb.X[0].view(np.int16)).view(torch.bfloat16).to(dev).view(T, h, d_h)
              for lb in wl.generate_layers(cfg, seed=0)]
    pipe = SelectionAttentionPipeline(T, h, d_h, cfg.tau, dev)
    res = []
    for overlap in (False, True, True):
        outs = [torch.zeros((T, h, d_h), dtype=torch.float32, device=dev) for _ in layers]
        pipe.run(layers, outs, overlap=overlap)
        torch.cuda.synchronize()
        res.append(outs)
    for a, b, c in zip(*res):
        assert torch.equal(a, b) and torch.equal(a, c)
        assert float(a.abs().max()) > 0.0
    assert ada.ada_device_status(pipe.sel)[0] == 0 and ada.ada_device_status(pipe.con)[0] == 0
    # against the oracle at the last layer: the chain of sets, then Eq. 2 with the device's map
    R = None
    for l, lb in enumerate(wl.generate_layers(cfg, seed=0)):
        X64 = wl.as_f64(lb.X[0])
        R = oracle.select_full(X64, cfg.tau)[0] if l == 0 else oracle.cascade_step(X64, cfg.tau, R).rep
    near = pipe.near[0].cpu().numpy()
    Xh = X64.reshape(T, h, d_h)
    ref = oracle.attention_reps(Xh, Xh, Xh, R, nearest_idx=near)
    assert np.max(np.abs(res[1][-1].cpu().numpy() - ref)) <= 2.0 ** -8 * float(np.max(np.abs(X64)))
    pipe.close()
