"""GPU parity of csp_decode_attn (Section 3.3: n-softmax decode attention over a pruned cache) against the
fp64 oracle, through the C interface.

Tolerance: the kernel computes the logits with bf16 x bf16 products accumulated in fp32 (exact products),
base-2 exponentials with about 2^-22 relative error, weights carried as a bf16 head plus a bf16 remainder
(2^-17 relative) and fp32 sums.  |gpu - oracle| <= 2e-3 * |oracle| + 1e-5 * max|v| covers it with a wide margin.
"""
import numpy as np
import pytest
import torch

from parity_util import bits  # noqa: F401  (shared helpers live next to the tests)

pytestmark = pytest.mark.gpu

REL, ABS = 2e-3, 1e-5


def _case(seed, B, Hq, Hkv, d, cap, rows=None, gain=1.0):
    g = torch.Generator().manual_seed(seed)
    q = (torch.randn(B, Hq, d, generator=g) * gain).to(torch.bfloat16)
    k = torch.randn(B, Hkv, cap, d, generator=g).to(torch.bfloat16)
    v = torch.randn(B, Hkv, cap, d, generator=g).to(torch.bfloat16)
    if rows is None:
        rows = torch.randint(0, cap + 1, (B, Hkv), generator=g, dtype=torch.int32)
    else:
        rows = torch.tensor(rows, dtype=torch.int32).reshape(B, Hkv)
    return q, k, v, rows


def _run(csp, oracle, q, k, v, rows, n=1.0, scale=0.0, poison=True):
    B, Hq, d = q.shape
    Hkv, cap = k.shape[1], k.shape[2]
    p = csp.Params(B, Hq, Hkv, d, 1, 0, cap, cap, n=n, scale=scale)
    po = oracle.Params(B, Hq, Hkv, d, 1, 0, cap, cap, dtype=oracle.BF16, n=n, scale=scale)
    want = oracle.decode_attn(po, q, k, v, rows.numpy())
    kd, vd = k.cuda(), v.cuda()
    if poison:      # rows past n_rows are unspecified: make them hostile
        for b in range(B):
            for h in range(Hkv):
                kd[b, h, int(rows[b, h]):] = float("nan")
                vd[b, h, int(rows[b, h]):] = float("inf")
    out = torch.full((B, Hq, d), 7.0, device="cuda")
    ws = csp.new_decode_workspace(p)
    csp.decode_attn(p, q.cuda(), kd, vd, rows.cuda(), out, ws)
    assert csp.device_status(ws) == 0
    got = out.cpu().numpy().astype(np.float64)
    tol = REL * np.abs(want) + ABS * float(v.float().abs().max())
    bad = np.abs(got - want) > tol
    assert not bad.any(), f"{bad.sum()} of {bad.size} outputs off; worst {np.abs(got - want).max()}"
    return got


@pytest.fixture(scope="module")
def csp():
    from paper_2412_04652_b200 import binding
    return binding


@pytest.mark.parametrize("G", [1, 2, 3, 4, 7, 8])
@pytest.mark.parametrize("d", [64, 128])
def test_decode_groups_and_head_dims(csp, oracle, G, d):
    q, k, v, rows = _case(100 + G + d, B=2, Hq=2 * G, Hkv=2, d=d, cap=333)
    _run(csp, oracle, q, k, v, rows)


def test_decode_ragged_tail_empty_and_full_heads(csp, oracle):
    q, k, v, rows = _case(7, B=1, Hq=8, Hkv=8, d=128, cap=200, rows=[0, 1, 15, 16, 17, 64, 199, 200])
    _run(csp, oracle, q, k, v, rows)


def test_decode_many_splits_and_many_units(csp, oracle):
    q, k, v, rows = _case(8, B=1, Hq=4, Hkv=1, d=128, cap=4096)          # one unit, 64 splits
    _run(csp, oracle, q, k, v, rows)
    q, k, v, rows = _case(9, B=40, Hq=16, Hkv=16, d=64, cap=130)         # 640 units, one split each
    _run(csp, oracle, q, k, v, rows)


@pytest.mark.parametrize("n", [0.0, 1.0, 50.0])
def test_decode_n_and_scale(csp, oracle, n):
    q, k, v, rows = _case(10, B=1, Hq=4, Hkv=2, d=128, cap=500, gain=3.0)
    a = _run(csp, oracle, q, k, v, rows, n=n)
    b = _run(csp, oracle, q, k, v, rows, n=n, scale=0.03)
    assert np.abs(a - b).max() > 1e-4          # the scale is really used


def test_decode_large_logits(csp, oracle):
    q, k, v, rows = _case(11, B=1, Hq=2, Hkv=2, d=128, cap=700, gain=12.0)   # logits of +-100: no overflow
    _run(csp, oracle, q, k, v, rows)


def test_decode_after_prune_uses_the_compacted_cache(csp, oracle):
    """The caches and row counts that csp_prune_layer leaves are what the decode step reads."""
    import csp_synth as synth
    from parity_util import GpuRun, gpu_params
    lays = [synth.interleaved_layout([200, 300, 200], 400), synth.interleaved_layout([150, 150, 100], 350)]
    cfg = synth.small_config("decode-after-prune", lays, 8, 4, 128, 32, 32, seed=5)
    q, k, v = synth.make_layer(cfg, 0, "cpu")[:3]
    p = gpu_params(csp, cfg)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets, cfg.total_budget).prune()
    assert run.status() == 0
    n_out = run.n_out.cpu()
    assert (n_out > 0).all()
    g = torch.Generator().manual_seed(3)
    q1 = torch.randn(cfg.batch, cfg.n_q_heads, cfg.head_dim, generator=g).to(torch.bfloat16)
    cap = p.out_capacity
    pd = csp.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, 1, 0, cap, cap)
    out = torch.zeros(cfg.batch, cfg.n_q_heads, cfg.head_dim, device="cuda")
    ws = csp.new_decode_workspace(pd)
    csp.decode_attn(pd, q1.cuda(), run.k_out, run.v_out, run.n_out, out, ws)
    assert csp.device_status(ws) == 0
    po = oracle.Params(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, 1, 0, cap, cap, dtype=oracle.BF16)
    ko, vo = run.k_out.cpu(), run.v_out.cpu()
    for b in range(cfg.batch):          # rows past n_out are unspecified on the GPU side: zero them for the oracle
        for h in range(cfg.n_kv_heads):
            ko[b, h, int(n_out[b, h]):] = 0
            vo[b, h, int(n_out[b, h]):] = 0
    want = oracle.decode_attn(po, q1, ko, vo, n_out.numpy())
    got = out.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want) <= REL * np.abs(want) + ABS * float(vo.float().abs().max())).all()


def test_decode_bad_row_count_is_flagged_and_host_errors(csp, oracle):
    q, k, v, rows = _case(12, B=1, Hq=2, Hkv=2, d=128, cap=100)
    p = csp.Params(1, 2, 2, 128, 1, 0, 100, 100)
    out = torch.zeros(1, 2, 128, device="cuda")
    ws = csp.new_decode_workspace(p)
    bad = torch.tensor([[101, 50]], dtype=torch.int32, device="cuda")
    csp.decode_attn(p, q.cuda(), k.cuda(), v.cuda(), bad, out, ws)
    assert csp.device_status(ws) & 8            # CSP_DEV_BAD_LEN; the row count was clamped to the capacity
    assert torch.isfinite(out).all()
    with pytest.raises(csp.CspError) as e:      # workspace too small
        csp.decode_attn(p, q.cuda(), k.cuda(), v.cuda(), rows.cuda(), out, ws[:256])
    assert e.value.code == 3
    p32 = csp.Params(1, 2, 2, 128, 1, 0, 100, 100, dtype=csp.F32)
    with pytest.raises(csp.CspError) as e:      # fp32 caches are not supported by this entry point
        csp.decode_attn(p32, q.cuda().float(), k.cuda().float(), v.cuda().float(), rows.cuda(), out, ws)
    assert e.value.code == 2
