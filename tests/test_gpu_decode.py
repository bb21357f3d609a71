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


# ------------------------------------------------------------------ Algorithm 1's iteration loop: csp_decode_step

def _score_tolerance_ok(got, want, what):
    """The score tolerance of the pruning pass: |gpu - oracle| <= 2e-3 |oracle| + 1e-6 max|oracle| per unit."""
    for u in range(want.shape[0]):
        w = want[u].astype(np.float64)
        tol = 2e-3 * np.abs(w) + 1e-6 * np.abs(w).max()
        bad = np.abs(got[u] - w) > tol
        assert not bad.any(), f"{what} unit {u}: {bad.sum()} of {w.size} sums off; worst {np.abs(got[u] - w).max()}"
        assert (got[u][w == 0.0] == 0.0).all(), f"{what} unit {u}: structural zeros must be exactly 0"


@pytest.mark.parametrize("Hq,Hkv,d,L0,steps,W", [(4, 2, 128, (700, 333), 40, 32), (7, 1, 64, (150,), 20, 16),
                                                 (8, 8, 128, (64, 1, 129, 40, 300, 77, 2, 500), 33, 32)])
def test_decode_steps_carry_the_scores_and_the_reprune_follows(csp, oracle, Hq, Hkv, d, L0, steps, W):
    """Tokens are appended one at a time to a cache of ragged per-sequence lengths; every step runs csp_decode_step.
    Checked: each step's attention output against the oracle; the running intra / inter sums against the oracle's
    (element by element) and against csp_score run from scratch on the final cache with the last W queries as the
    window; then csp_select on the carried sums is the exact selection for those sums and agrees with the
    selection from the from-scratch scores except at boundary ties."""
    B, G = len(L0), Hq // Hkv
    cap = max(L0) + steps
    gen = torch.Generator().manual_seed(7 * Hq + steps)
    k = torch.randn(B, Hkv, cap, d, generator=gen).to(torch.bfloat16)
    v = torch.randn(B, Hkv, cap, d, generator=gen).to(torch.bfloat16)
    mod = (torch.rand(B, Hkv, cap, generator=gen) < 0.5).to(torch.uint8)          # labels differ per head after a prune
    qs = (torch.randn(steps, B, Hq, d, generator=gen) * 1.5).to(torch.bfloat16)
    new_label = (torch.rand(steps, B, generator=gen) < 0.3).to(torch.uint8)        # some appended tokens are visual
    for b in range(B):                                                              # appended rows carry their token's label
        for i in range(steps):
            mod[b, :, L0[b] + i] = new_label[i, b]
    p = csp.Params(B, Hq, Hkv, d, 1, 0, cap, cap)
    po = oracle.Params(B, Hq, Hkv, d, 1, 0, cap, cap, dtype=oracle.BF16)
    kd, vd, modd = k.cuda(), v.cuda(), mod.cuda()
    for b in range(B):                               # rows not yet appended are unspecified: make them hostile
        kd[b, :, L0[b]:] = float("nan")
        vd[b, :, L0[b]:] = float("inf")
    acc_s = torch.full((B, Hkv, cap), 9.0, device="cuda")
    acc_c = torch.full((B, Hkv, cap), -9.0, device="cuda")
    o_s, o_c = np.full((B, Hkv, cap), 9.0), np.full((B, Hkv, cap), -9.0)
    out = torch.zeros(B, Hq, d, device="cuda")
    ws = csp.new_decode_step_workspace(p)
    for i in range(steps):
        rows = torch.tensor([[L0[b] + i + 1] * Hkv for b in range(B)], dtype=torch.int32)
        for b in range(B):                           # the new token's K and V rows enter the cache first
            kd[b, :, L0[b] + i] = k[b, :, L0[b] + i].cuda()
            vd[b, :, L0[b] + i] = v[b, :, L0[b] + i].cuda()
        first = i == steps - W
        csp.decode_step(p, qs[i].cuda(), kd, vd, rows.cuda(), modd, new_label[i].cuda(), first, out, acc_s, acc_c, ws)
        want = oracle.decode_step(po, qs[i], k, v, rows.numpy(), mod.numpy(), new_label[i].numpy(), o_s, o_c, first)
        if i % 7 == 0 or i == steps - 1:
            got = out.cpu().numpy().astype(np.float64)
            tol = REL * np.abs(want) + ABS * float(v.float().abs().max())
            assert (np.abs(got - want) <= tol).all(), f"step {i}: attention output off by {np.abs(got - want).max()}"
    assert csp.device_status(ws) == 0
    g_s, g_c = acc_s.cpu().numpy(), acc_c.cpu().numpy()
    _score_tolerance_ok(g_s.reshape(B * Hkv, cap), o_s.reshape(B * Hkv, cap), "intra")
    _score_tolerance_ok(g_c.reshape(B * Hkv, cap), o_c.reshape(B * Hkv, cap), "inter")

    # from scratch on the final cache: the last W queries are the observation window
    lens = torch.tensor([L0[b] + steps for b in range(B)], dtype=torch.int32)
    R = W
    q_win = qs[steps - W:].permute(1, 2, 0, 3).contiguous()                        # [B, Hq, W, d]
    ps = csp.Params(B, Hq, Hkv, d, W, R, cap, cap)
    ss = torch.zeros(B, Hkv, cap, device="cuda")
    sc = torch.zeros(B, Hkv, cap, device="cuda")
    wsp = csp.new_workspace(ps)
    csp.score(ps, q_win.cuda(), kd, modd, lens.cuda(), ss, sc, wsp)
    assert csp.device_status(wsp) == 0
    for b in range(B):
        N = int(lens[b]) - R
        if N <= 0:
            continue
        _score_tolerance_ok(g_s[b, :, :N], ss[b, :, :N].cpu().numpy(), "carried vs from-scratch intra")
        _score_tolerance_ok(g_c[b, :, :N], sc[b, :, :N].cpu().numpy(), "carried vs from-scratch inter")

    # the prune that follows: Eq. 2-4 on the carried sums
    bud = torch.tensor([[max(1, (L0[b] + steps) // 9), 5, 3, max(1, (L0[b] + steps) // 7)] for b in range(B)], dtype=torch.int32)
    idx = torch.full((B, Hkv, cap), -1, dtype=torch.int32, device="cuda")
    n_out = torch.zeros(B, Hkv, dtype=torch.int32, device="cuda")
    csp.select(ps, acc_s, acc_c, modd, lens.cuda(), bud.cuda(), idx, n_out, wsp)
    assert csp.device_status(wsp) & ~csp.DEV_K_CLAMPED == 0
    pos = oracle.Params(B, Hq, Hkv, d, W, R, cap, cap, dtype=oracle.BF16)
    i_ref, n_ref, _, _ = oracle.select(pos, g_s, g_c, mod.numpy(), lens.numpy(), bud.numpy())
    np.testing.assert_array_equal(n_out.cpu().numpy(), n_ref)
    for b in range(B):
        for h in range(Hkv):
            n = int(n_ref[b, h])
            np.testing.assert_array_equal(idx[b, h, :n].cpu().numpy(), i_ref[b, h, :n])
    k_out, v_out = torch.zeros_like(kd), torch.zeros_like(vd)
    mod_out = torch.zeros_like(modd)
    csp.compact(ps, kd, vd, modd, idx, n_out, k_out, v_out, mod_out)
    for b in range(B):
        for h in range(Hkv):
            n = int(n_ref[b, h])
            ii = i_ref[b, h, :n]
            np.testing.assert_array_equal(bits(k_out[b, h, :n]), bits(k)[b, h][ii])
            np.testing.assert_array_equal(bits(v_out[b, h, :n]), bits(v)[b, h][ii])
            np.testing.assert_array_equal(mod_out[b, h, :n].cpu().numpy(), mod[b, h].numpy()[ii])


def test_decode_step_bad_row_counts_are_clamped_and_flagged(csp, oracle):
    q, k, v, rows = _case(71, 2, 4, 2, 128, 90, rows=[[90, 40], [13, 64]])
    bad = rows.clone()
    bad[0, 0], bad[1, 0] = 500, -7                    # above the capacity, negative
    p = csp.Params(2, 4, 2, 128, 1, 0, 90, 90)
    mod = torch.zeros(2, 2, 90, dtype=torch.uint8, device="cuda")
    lab = torch.zeros(2, dtype=torch.uint8, device="cuda")
    acc_s, acc_c = torch.full((2, 2, 90), 3.0, device="cuda"), torch.full((2, 2, 90), 3.0, device="cuda")
    out = torch.zeros(2, 4, 128, device="cuda")
    ws = csp.new_decode_step_workspace(p)
    csp.decode_step(p, q.cuda(), k.cuda(), v.cuda(), bad.cuda(), mod, lab, True, out, acc_s, acc_c, ws)
    assert csp.device_status(ws) & csp.DEV_BAD_LEN
    po = oracle.Params(2, 4, 2, 128, 1, 0, 90, 90, dtype=oracle.BF16)
    clamped = torch.tensor([[90, 40], [0, 64]], dtype=torch.int32)
    o_s, o_c = np.zeros((2, 2, 90)), np.zeros((2, 2, 90))
    want = oracle.decode_step(po, q, k, v, clamped.numpy(), mod.cpu().numpy(), lab.cpu().numpy(), o_s, o_c, True)
    got = out.cpu().numpy().astype(np.float64)
    assert (np.abs(got - want) <= REL * np.abs(want) + ABS * float(v.float().abs().max())).all()
    _score_tolerance_ok(acc_s.cpu().numpy().reshape(4, 90), o_s.reshape(4, 90), "intra")
    assert (acc_c == 0).all() and (acc_s[1, 0] == 0).all()       # a unit without rows: its sums are cleared


def test_decode_step_rejects_bad_arguments(csp):
    p = csp.Params(1, 2, 2, 128, 1, 0, 64, 64)
    z = torch.zeros(1, 2, 64, 128, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(1, 2, 128, dtype=torch.bfloat16, device="cuda")
    rows = torch.zeros(1, 2, dtype=torch.int32, device="cuda")
    mod = torch.zeros(1, 2, 64, dtype=torch.uint8, device="cuda")
    lab = torch.zeros(1, dtype=torch.uint8, device="cuda")
    acc = torch.zeros(1, 2, 64, device="cuda")
    out = torch.zeros(1, 2, 128, device="cuda")
    small = csp.new_decode_workspace(p)              # the workspace of the plain decode call is too small
    with pytest.raises(csp.CspError) as e:
        csp.decode_step(p, q, z, z, rows, mod, lab, True, out, acc, acc.clone(), small)
    assert e.value.code == csp.ERR_WORKSPACE
    ws = csp.new_decode_step_workspace(p)
    csp.decode_step(p, q, z, z, rows, mod, lab, True, out, acc, acc.clone(), ws)     # zero rows: zeros everywhere
    assert csp.device_status(ws) == 0 and (out == 0).all() and (acc == 0).all()
