"""GPU parity: the CUDA library against the CPU oracle, element by element, on the same seeded
inputs, through the C interface.  Sizes span several 128-key tiles and ragged tails."""
import numpy as np
import pytest
import torch

import csp_synth as synth
from parity_util import (GpuRun, assert_compaction_exact, assert_index_sets_match,
                         assert_selection_follows_own_scores, assert_scores_close, bits, gpu_params, orc_params)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def csp():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2412_04652_b200 import binding
    binding.lib()
    return binding


def _layout(L, n_img, img_len, seed):
    rng = np.random.RandomState(seed)
    img_len = max(1, min(img_len, (L - 40) // n_img))
    text = L - n_img * img_len
    assert text >= 40
    cuts = np.sort(rng.randint(0, text - 40 + 1, size=n_img))
    spans = np.diff(np.concatenate([[0], cuts, [text - 40]])).tolist()
    spans[-1] += 40
    return synth.interleaved_layout(spans, img_len)


def _case(lens, n_q, n_kv, d, W, R, dtype=torch.bfloat16, seed=0, img=(2, 50), **kw):
    lays = [_layout(L, img[0], img[1], seed + i) for i, L in enumerate(lens)]
    return synth.small_config("case", lays, n_q, n_kv, d, W, R, dtype=dtype, seed=seed, **kw)


def _run_score(csp, oracle, cfg, modality=None, gpu_kw=None, orc_kw=None, q_gain=1.0, lse=None):
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    if q_gain != 1.0:
        q = (q.float() * q_gain).to(cfg.dtype)
    mod = cfg.modality() if modality is None else modality
    p = gpu_params(csp, cfg, **(gpu_kw or {}))
    run = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, cfg.budgets, lse=lse).score()
    assert run.status() == 0
    op = orc_params(oracle, cfg, **(orc_kw or {}))
    s, c = oracle.score(op, q.cpu(), k.cpu(), mod, cfg.seq_lens, lse=lse)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent, "self")
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent, "cross")
    return run, s, c


# ------------------------------------------------------------------ score

@pytest.mark.parametrize("lens,n_q,n_kv,d,W,R,dtype", [
    ((300,), 2, 2, 128, 32, 32, torch.bfloat16),            # MHA, 3 tiles, ragged tail
    ((517, 130, 1029), 4, 4, 128, 32, 32, torch.bfloat16),  # ragged batch
    ((700,), 4, 2, 128, 32, 32, torch.bfloat16),            # GQA G=2
    ((700, 257), 12, 4, 128, 32, 32, torch.bfloat16),       # G=3
    ((390,), 4, 1, 128, 32, 32, torch.bfloat16),            # G=4
    ((450,), 5, 1, 64, 32, 32, torch.bfloat16),             # G=5, 128-byte rows
    ((1300, 640), 7, 1, 128, 32, 32, torch.bfloat16),       # G=7 (the GQA benchmark shape)
    ((333,), 8, 1, 128, 16, 16, torch.bfloat16),            # G=8, narrow window
    ((1024,), 4, 4, 64, 16, 16, torch.float32),             # fp32 (3xTF32)
    ((500,), 4, 2, 128, 32, 32, torch.float32),             # fp32, 512-byte rows, G=2
    ((400,), 2, 2, 256, 32, 32, torch.bfloat16),            # 512-byte bf16 rows
    ((260,), 2, 2, 128, 5, 9, torch.bfloat16),              # odd window, R > W
    ((260,), 2, 2, 128, 32, 7, torch.bfloat16),             # R < W: causal mask cuts into candidates
    ((129,), 1, 1, 128, 32, 0, torch.bfloat16),             # R = 0
    ((128,), 2, 2, 128, 32, 32, torch.bfloat16),            # exactly one tile
    ((64,), 2, 2, 128, 32, 32, torch.bfloat16),             # less than a tile
])
def test_score_matches_oracle(csp, oracle, lens, n_q, n_kv, d, W, R, dtype):
    _run_score(csp, oracle, _case(lens, n_q, n_kv, d, W, R, dtype=dtype, seed=len(lens) + n_q))


@pytest.mark.parametrize("lens_hi,n_seq,heads,d", [(1000, 40, 8, 128), (2500, 20, 16, 128), (1800, 40, 8, 64),
                                                    (5000, 10, 32, 64)])
def test_score_many_units_resident_clusters(csp, oracle, lens_hi, n_seq, heads, d):
    """More MHA units than clusters fit on the GPU: the resident-cluster kernel walks unit after unit
    (clusters of 1, 2 and 4 CTAs; 256- and 128-byte rows), ragged lengths, every unit compared."""
    rng = np.random.RandomState(lens_hi)
    lens = tuple(int(x) for x in rng.randint(90, lens_hi, size=n_seq))
    cfg = _case(lens, heads, heads, d, 32, 32, seed=17)
    mod = cfg.modality()
    mod[:, -40:] = (rng.rand(n_seq, 40) < 0.3)          # padding labels and some mixed windows
    for b, L in enumerate(lens):
        mod[b, L - 32:L] = (rng.rand(32) < (0.5 if b % 3 == 0 else 0.0))
    _run_score(csp, oracle, cfg, modality=mod.astype(np.uint8))


@pytest.mark.parametrize("later_gain", [6.0, 0.05])
def test_score_resident_clusters_logits_far_from_the_first_tile(csp, oracle, later_gain):
    """Keys after a unit's first tile are scaled so that the largest logits sit about 60 nats above (or far
    below) those of the first tile: the running reference of the resident-cluster kernel has to follow."""
    rng = np.random.RandomState(3)
    lens = tuple(int(x) for x in rng.randint(200, 900, size=40))
    cfg = _case(lens, 8, 8, 128, 32, 32, seed=23)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    q = (q.float() * 3.0).to(cfg.dtype)
    k = k.clone()
    k[:, :, 128:] = (k[:, :, 128:].float() * later_gain).to(cfg.dtype)
    p = gpu_params(csp, cfg)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets).score()
    assert run.status() == 0
    s, c = oracle.score(orc_params(oracle, cfg), q.cpu(), k.cpu(), cfg.modality(), cfg.seq_lens)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent, "self")
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent, "cross")


def test_score_mixed_modality_window_and_per_head_labels(csp, oracle):
    cfg = _case((600, 350), 4, 2, 128, 32, 32, seed=5)
    rng = np.random.RandomState(0)
    mod = (rng.rand(2, 2, cfg.max_len) < 0.5).astype(np.uint8)      # per head, random incl. the window
    _run_score(csp, oracle, cfg, modality=mod)
    mod3 = (rng.randint(0, 3, size=(2, cfg.max_len))).astype(np.uint8)  # three labels
    _run_score(csp, oracle, cfg, modality=mod3)


@pytest.mark.parametrize("n", [0.0, 1.0, 100.0])
def test_score_n_sensitive(csp, oracle, n):
    # logits ~ 8 * N(0,1) - 20: the exponential mass is comparable to or far below n
    cfg = _case((200, 64), 2, 2, 128, 32, 32, seed=7)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    q = (q.float() * 8).to(cfg.dtype)
    q[..., 0] = 1.0
    k[..., 0] = -20.0 * np.sqrt(128)
    p = gpu_params(csp, cfg, n=n)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets).score()
    assert run.status() == 0
    s, c = oracle.score(orc_params(oracle, cfg, n=n), q.cpu(), k.cpu(), cfg.modality(), cfg.seq_lens)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent)


def test_score_large_logits_and_explicit_scale(csp, oracle):
    cfg = _case((300,), 2, 2, 128, 32, 32, seed=8)
    _run_score(csp, oracle, cfg, q_gain=6.0)
    _run_score(csp, oracle, cfg, gpu_kw=dict(scale=0.25), orc_kw=dict(scale=0.25))


def test_score_all_zero_queries_closed_form(csp, oracle):
    cfg = _case((300,), 2, 2, 128, 32, 32, seed=9)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    q.zero_()
    mod = cfg.modality()
    run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod, cfg.seq_lens, cfg.budgets).score()
    L, W = 300, 32
    want = sum(1.0 / (1.0 + (L - W + w) + 1) for w in range(W))   # every window row is text here
    s, c = run.ss.cpu().numpy()[0, 0, :L - 32], run.sc.cpu().numpy()[0, 0, :L - 32]
    text = mod[0, :L - 32] == 0
    np.testing.assert_allclose(s[text], want, rtol=1e-5)
    np.testing.assert_allclose(c[~text], want, rtol=1e-5)
    assert (s[~text] == 0).all() and (c[text] == 0).all()


def test_score_with_supplied_lse(csp, oracle):
    cfg = _case((500, 200), 4, 2, 128, 32, 32, seed=10)
    q, k, v = synth.make_layer(cfg, 0, "cpu")
    G = 2
    lse = np.zeros((2, 4, 32))
    for b in range(2):
        L = int(cfg.seq_lens[b])
        for hq in range(4):
            o = (q[b, hq].double() @ k[b, hq // G, :L].double().T / np.sqrt(128)).numpy()
            for w in range(32):
                lse[b, hq, w] = np.log(np.exp(o[w, :L - 32 + w + 1]).sum())
    p = gpu_params(csp, cfg)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets, lse=lse).score()
    s, c = oracle.score(orc_params(oracle, cfg), q, k, cfg.modality(), cfg.seq_lens)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent)


@pytest.mark.parametrize("lens_hi,n_seq,heads,d", [(1000, 40, 8, 128), (2500, 20, 16, 64)])
def test_score_with_supplied_lse_many_units(csp, oracle, lens_hi, n_seq, heads, d):
    """Many MHA units with the rows' log-sum-exp supplied: the resident-cluster kernel without its first pass
    (clusters of 1 and 2).  The oracle computes its own normaliser; the results must agree."""
    rng = np.random.RandomState(lens_hi + 1)
    lens = tuple(int(x) for x in rng.randint(90, lens_hi, size=n_seq))
    cfg = _case(lens, heads, heads, d, 32, 32, seed=19)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    lse = np.zeros((n_seq, heads, 32))
    for b, L in enumerate(lens):
        o = torch.einsum("hwd,htd->hwt", q[b].double(), k[b, :, :L].double()) / np.sqrt(d)
        pos = L - 32 + torch.arange(32, device="cuda")
        o.masked_fill_((torch.arange(L, device="cuda")[None, :] > pos[:, None])[None], float("-inf"))
        lse[b] = torch.logsumexp(o, dim=2).cpu().numpy()
    mod = cfg.modality()
    for b, L in enumerate(lens):
        mod[b, L - 32:L] = (rng.rand(32) < (0.5 if b % 3 == 0 else 0.0))          # some mixed windows
    run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod, cfg.seq_lens, cfg.budgets, lse=lse).score()
    assert run.status() == 0
    s, c = oracle.score(orc_params(oracle, cfg), q.cpu(), k.cpu(), mod, cfg.seq_lens)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent, "self")
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent, "cross")
    plain = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod, cfg.seq_lens, cfg.budgets).score()
    for b, L in enumerate(lens):                         # and against the two-pass run of the same kernel
        np.testing.assert_allclose(run.ss[b, :, :L - 32].cpu().numpy(), plain.ss[b, :, :L - 32].cpu().numpy(), rtol=1e-4, atol=1e-9)


def test_score_mean_over_all_heads(csp, oracle):
    cfg = _case((420, 300), 8, 4, 128, 32, 32, seed=11)
    _run_score(csp, oracle, cfg, gpu_kw=dict(head_reduce=csp.HEADS_MEAN_ALL),
               orc_kw=dict(head_reduce=oracle.HEADS_MEAN_ALL))


def test_score_strided_views_and_padding_ignored(csp, oracle):
    cfg = _case((300, 200), 4, 2, 128, 32, 32, seed=12)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    big = torch.full((2, 2, cfg.max_len + 24, 256), float("nan"), dtype=k.dtype, device="cuda")
    big[:, :, 8:8 + cfg.max_len, 128:] = k
    kview = big[:, :, 8:8 + cfg.max_len, 128:]
    kview[1, :, 200:] = float("nan")                      # padding rows hold NaN
    p = gpu_params(csp, cfg)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets)
    run.k = kview
    run.score()
    assert run.status() == 0
    s, c = oracle.score(orc_params(oracle, cfg), q.cpu(), k.cpu(), cfg.modality(), cfg.seq_lens)
    assert_scores_close(run.ss.cpu().numpy(), s, cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), c, cfg.seq_lens, cfg.recent)


def test_score_is_bit_reproducible(csp, oracle):
    cfg = _case((900, 400), 7, 1, 128, 32, 32, seed=13)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    runs = [GpuRun(csp, gpu_params(csp, cfg), q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets).score()
            for _ in range(2)]
    for b, L in enumerate(cfg.seq_lens):
        assert torch.equal(runs[0].ss[b, :, :L - 32], runs[1].ss[b, :, :L - 32])
        assert torch.equal(runs[0].sc[b, :, :L - 32], runs[1].sc[b, :, :L - 32])


# ------------------------------------------------------------------ select (bit-exact on equal fp32 scores)

def _select_case(csp, oracle, B, H, lens, R, budgets, quantise=None, seed=0, total=None, cap=None, **mode):
    rng = np.random.RandomState(seed)
    Lm = max(lens)
    s = rng.rand(B, H, Lm).astype(np.float32)
    c = rng.rand(B, H, Lm).astype(np.float32)
    if quantise:
        s, c = np.floor(s * quantise) / quantise, np.floor(c * quantise) / quantise
    mod = (rng.rand(B, Lm) < 0.6).astype(np.uint8)
    cap = cap if cap is not None else Lm
    kw = dict(combine=mode.get("combine", 0), select_mode=mode.get("select_mode", 0))
    p = csp.Params(B, H, H, 128, min(32, min(lens)) if min(lens) > 0 else 1, R, Lm, cap, **kw)
    dummy = torch.zeros(B, H, 1, 128, dtype=torch.bfloat16)
    run = GpuRun(csp, p, dummy, dummy, dummy, mod, lens, budgets, total_budget=total)
    run.ss, run.sc = torch.from_numpy(s).cuda(), torch.from_numpy(c).cuda()
    run.select()
    op = oracle.Params(B, H, H, 128, p.window, R, Lm, cap, **kw)
    idx, n_out, flags, _ = oracle.select(op, s, c, mod, np.array(lens, np.int32), np.array(budgets, np.int32),
                                         None if total is None else np.array(total, np.int32))
    gi, gn = run.idx.cpu().numpy(), run.n_out.cpu().numpy()
    np.testing.assert_array_equal(gn, n_out)
    for b in range(B):
        for h in range(H):
            n = n_out[b, h]
            if n > 0:
                np.testing.assert_array_equal(gi[b, h, :n], idx[b, h, :n])
    return run.status(), flags


@pytest.mark.parametrize("mode", [dict(), dict(combine=1), dict(select_mode=1), dict(select_mode=1, combine=1),
                                  dict(select_mode=2), dict(select_mode=2, combine=1)])
def test_select_matches_oracle_exactly(csp, oracle, mode):
    lens = (3000, 1500, 777)
    nb = {0: 4, 1: 2, 2: 1}[mode.get("select_mode", 0)]
    budgets = np.random.RandomState(1).randint(0, 400, size=(3, nb))
    _select_case(csp, oracle, 3, 2, lens, 32, budgets, seed=1, **mode)
    _select_case(csp, oracle, 3, 2, lens, 32, budgets, quantise=16, seed=2, **mode)   # heavy ties


@pytest.mark.parametrize("lens", [(500, 300, 77), (512, 33), (1000, 513, 64), (1024,), (2048, 1500, 1025), (1300, 40)])
@pytest.mark.parametrize("mode", [dict(), dict(combine=1), dict(select_mode=1), dict(select_mode=2)])
def test_select_short_caches(csp, oracle, lens, mode):
    """Caches of up to 512, 1024 and 2048 positions take smaller CTAs (the re-prune rounds of a serving batch)."""
    nb = {0: 4, 1: 2, 2: 1}[mode.get("select_mode", 0)]
    B = len(lens)
    budgets = np.random.RandomState(len(lens) + lens[0]).randint(0, max(lens) // 4, size=(B, nb))
    _select_case(csp, oracle, B, 3, lens, 32, budgets, seed=21, **mode)
    _select_case(csp, oracle, B, 3, lens, 32, budgets, quantise=8, seed=22, **mode)       # heavy ties
    _select_case(csp, oracle, B, 40, lens, 5, budgets, quantise=64, seed=23, **mode)      # many units


def test_select_all_equal_scores_and_extreme_budgets(csp, oracle):
    lens = (2100, 40)
    st, flags = _select_case(csp, oracle, 2, 1, lens, 8, [[5, 7, 0, 0], [0, 0, 0, 0]], quantise=1, seed=3)
    assert st == 0
    st, flags = _select_case(csp, oracle, 2, 1, lens, 8, [[100000, 100000, 3, -4], [1, 1, 1, 1]], seed=4)
    assert st == csp.DEV_K_CLAMPED and (flags[0] & oracle.FLAG_K_CLAMPED).all()


def test_select_identity_capacity_and_short_sequences(csp, oracle):
    st, flags = _select_case(csp, oracle, 3, 2, (500, 20, 0), 32, [[10, 10, 10, 10]] * 3, seed=5, total=[501, 0, 0])
    assert st == 0 and (flags & oracle.FLAG_IDENTITY).all()
    st, flags = _select_case(csp, oracle, 2, 1, (500, 300), 32, [[40, 40, 40, 40], [2, 2, 2, 2]], seed=6, cap=64)
    assert st == csp.DEV_CAPACITY and (flags[0] & oracle.FLAG_CAPACITY).all() and not flags[1].any()


def test_select_long_sequence(csp, oracle):
    _select_case(csp, oracle, 1, 2, (32768,), 32, [[1626, 0, 0, 4301]], seed=7)
    _select_case(csp, oracle, 1, 1, (32768,), 32, [[1626, 3, 9, 4301]], quantise=64, seed=8)


def test_select_overall_mode_long_caches(csp, oracle):
    """One top-K on s + c (the ablation's comparison arm), through every selection kernel shape."""
    _select_case(csp, oracle, 2, 2, (32768, 9000), 32, [[4000], [100000]], seed=12, select_mode=2)
    _select_case(csp, oracle, 1, 1, (66000,), 32, [[700]], quantise=32, seed=13, select_mode=2)
    _select_case(csp, oracle, 40, 8, tuple(3000 + 13 * i for i in range(40)), 32, [[300 + i] for i in range(40)],
                 quantise=64, seed=14, select_mode=2)


def test_select_cache_longer_than_cluster_limit(csp, oracle):
    """Above 65536 positions the one-CTA-per-unit kernel takes over (keys partly staged in shared memory)."""
    _select_case(csp, oracle, 1, 2, (70001,), 32, [[3000, 11, 0, 9000]], seed=10)
    _select_case(csp, oracle, 1, 1, (66000,), 32, [[500, 500, 500, 500]], quantise=32, seed=11)


def test_select_negative_and_signed_zero_scores(csp, oracle):
    rng = np.random.RandomState(9)
    s = rng.randn(1, 1, 700).astype(np.float32)
    s[0, 0, ::7] = 0.0
    s[0, 0, 3::7] = -0.0
    c = -s
    mod = np.zeros((1, 700), np.uint8)
    p = csp.Params(1, 1, 1, 128, 32, 32, 700, 700, select_mode=1)
    dummy = torch.zeros(1, 1, 1, 128, dtype=torch.bfloat16)
    run = GpuRun(csp, p, dummy, dummy, dummy, mod, [700], [[300, 250]])
    run.ss, run.sc = torch.from_numpy(s).cuda(), torch.from_numpy(c).cuda()
    run.select()
    idx, n_out, _, _ = oracle.select(oracle.Params(1, 1, 1, 128, 32, 32, 700, 700, select_mode=1), s, c, mod,
                                     np.array([700], np.int32), np.array([[300, 250]], np.int32))
    n = int(n_out[0, 0])
    assert int(run.n_out[0, 0]) == n
    np.testing.assert_array_equal(run.idx.cpu().numpy()[0, 0, :n], idx[0, 0, :n])


# ------------------------------------------------------------------ compact

def test_compact_is_bit_exact_with_strides(csp, oracle):
    cfg = _case((400, 250), 4, 2, 128, 32, 32, seed=20)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    p = gpu_params(csp, cfg, cap=300)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets)
    rng = np.random.RandomState(0)
    idx = np.full((2, 2, 300), -1, np.int32)
    n_out = np.array([[300, 17], [0, -1]], np.int32)
    for b in range(2):
        for h in range(2):
            n = max(int(n_out[b, h]), 0)
            idx[b, h, :n] = np.sort(rng.choice(int(cfg.seq_lens[b]), n, replace=False))
    run.idx, run.n_out = torch.from_numpy(idx).cuda(), torch.from_numpy(n_out).cuda()
    wide = torch.zeros(2, 2, 300, 256, dtype=k.dtype, device="cuda")
    run.k_out = wide[..., :128]
    run.v_out = wide[..., 128:]
    run.compact()
    assert_compaction_exact(run, cfg.modality())
    ko, vo, mo = oracle.compact(orc_params(oracle, cfg, cap=300), k.cpu(), v.cpu(), cfg.modality(), idx, n_out)
    np.testing.assert_array_equal(bits(run.k_out), ko)
    np.testing.assert_array_equal(bits(run.v_out), vo)
    np.testing.assert_array_equal(run.mod_out.cpu().numpy(), mo)


def test_compact_row_count_above_capacity_is_clamped_not_faulted(csp, oracle):
    """n_out is caller-supplied device data for csp_compact: a count above out_capacity copies the first
    out_capacity rows and touches nothing behind the unit (canary rows, the next unit's rows, labels)."""
    cfg = _case((400, 250), 4, 2, 128, 32, 32, seed=24)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    cap = 70                                              # not a multiple of the 64 / 128 rows a CTA covers
    p = gpu_params(csp, cfg, cap=cap)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets)
    rng = np.random.RandomState(2)
    idx = np.zeros((2, 2, cap), np.int32)
    for b in range(2):
        for h in range(2):
            idx[b, h] = np.sort(rng.choice(int(cfg.seq_lens[b]), cap, replace=False))
    n_out = np.array([[cap + 5, cap], [cap + 1000, 3]], np.int32)
    run.idx, run.n_out = torch.from_numpy(idx).cuda(), torch.from_numpy(n_out).cuda()
    canary = 0x7F7F
    big_k = torch.full((2, 2, cap + 8, 128), 0, dtype=torch.int16, device="cuda") + canary
    big_v = big_k.clone()
    big_m = torch.full((2 * 2 * cap + 64,), 0xEE, dtype=torch.uint8, device="cuda")
    run.k_out, run.v_out = big_k.view(torch.bfloat16)[:, :, :cap], big_v.view(torch.bfloat16)[:, :, :cap]
    run.mod_out = big_m[:2 * 2 * cap].view(2, 2, cap)
    run.compact()
    torch.cuda.synchronize()
    assert (big_k[:, :, cap:] == canary).all() and (big_v[:, :, cap:] == canary).all()
    assert (big_m[2 * 2 * cap:] == 0xEE).all()
    kb, vb = bits(k), bits(v)
    for b in range(2):
        for h in range(2):
            n = min(int(n_out[b, h]), cap)
            np.testing.assert_array_equal(bits(run.k_out[b, h, :n]), kb[b, h][idx[b, h, :n]])
            np.testing.assert_array_equal(bits(run.v_out[b, h, :n]), vb[b, h][idx[b, h, :n]])
            np.testing.assert_array_equal(run.mod_out[b, h, :n].cpu().numpy(), cfg.modality()[b][idx[b, h, :n]])
    assert (big_k[1, 1, 3:] == canary).all()              # the short unit wrote its three rows only


@pytest.mark.parametrize("d,dtype", [(128, torch.bfloat16), (64, torch.bfloat16), (64, torch.float32)])
def test_compact_in_place_matches_out_of_place(csp, oracle, d, dtype):
    """k_out is k and v_out is v: rows move down inside the cache.  Dense keeps (many rows shifting by a few
    positions, across several 128-row chunks) are the hazardous case; an identity prefix and empty units too."""
    lens = (1500, 700, 333)
    cfg = _case(lens, 4, 2, d, 16, 16, dtype=dtype, seed=21)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    cap = 1500
    p = gpu_params(csp, cfg, cap=cap)
    rng = np.random.RandomState(1)
    idx = np.full((3, 2, cap), -1, np.int32)
    n_out = np.array([[1490, 600], [700, 0], [129, 1]], np.int32)      # near-full, sparse, identity, empty, chunk + 1, one
    for b in range(3):
        for h in range(2):
            n = int(n_out[b, h])
            idx[b, h, :n] = np.sort(rng.choice(lens[b], n, replace=False))
    idx[0, 1, :200] = np.arange(200)                                    # identity prefix, then a jump
    idx[0, 1, 200:600] = np.sort(rng.choice(np.arange(200, lens[0]), 400, replace=False))
    ko, vo, mo = oracle.compact(orc_params(oracle, cfg, cap=cap), k.cpu(), v.cpu(), cfg.modality(), idx, n_out)
    if ko.dtype == np.float32:
        ko, vo = ko.view(np.uint32), vo.view(np.uint32)
    run = GpuRun(csp, p, q, k.clone(), v.clone(), cfg.modality(), cfg.seq_lens, cfg.budgets)
    run.idx, run.n_out = torch.from_numpy(idx).cuda(), torch.from_numpy(n_out).cuda()
    run.k_out, run.v_out = run.k, run.v                                 # the same tensors
    run.compact()
    kb, vb = bits(run.k), bits(run.v)
    for b in range(3):
        for h in range(2):
            n = int(n_out[b, h])
            np.testing.assert_array_equal(kb[b, h, :n], ko[b, h, :n])
            np.testing.assert_array_equal(vb[b, h, :n], vo[b, h, :n])
            np.testing.assert_array_equal(run.mod_out.cpu().numpy()[b, h, :n], mo[b, h, :n])
            if n == 0:                                                  # an empty unit is left untouched
                np.testing.assert_array_equal(kb[b, h, :lens[b]], bits(k)[b, h, :lens[b]])
    # only one of the two tensors in place is refused
    run2 = GpuRun(csp, p, q, k.clone(), v.clone(), cfg.modality(), cfg.seq_lens, cfg.budgets)
    run2.idx, run2.n_out = run.idx, run.n_out
    run2.k_out = run2.k
    with pytest.raises(csp.CspError) as e:
        run2.compact()
    assert e.value.code == 2


def test_prune_layer_in_place(csp, oracle):
    """Algorithm 1 without a second cache buffer: k_out / v_out are the input tensors."""
    cfg = _case((1200, 640), 8, 4, 128, 32, 32, seed=22)
    run, ref = _run_prune(csp, oracle, cfg)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    p = gpu_params(csp, cfg)
    inp = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets, total_budget=cfg.total_budget)
    inp.k_out, inp.v_out = inp.k, inp.v
    inp.prune()
    assert inp.status() == 0
    assert torch.equal(inp.n_out, run.n_out) and torch.equal(inp.idx, run.idx)
    n_out = run.n_out.cpu().numpy()
    for b in range(cfg.batch):
        for h in range(cfg.n_kv_heads):
            n = int(n_out[b, h])
            assert torch.equal(inp.k[b, h, :n], run.k_out[b, h, :n]) and torch.equal(inp.v[b, h, :n], run.v_out[b, h, :n])
    assert torch.equal(inp.mod_out, run.mod_out)


# ------------------------------------------------------------------ Algorithm 1 end to end

def _run_prune(csp, oracle, cfg, layer=0, with_optional=True, **mode):
    q, k, v = synth.make_layer(cfg, layer, "cuda")
    p = gpu_params(csp, cfg, **mode)
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets, total_budget=cfg.total_budget)
    run.prune(with_optional)
    ref = oracle.prune_layer(orc_params(oracle, cfg, **mode), q.cpu(), k.cpu(), v.cpu(), cfg.modality(),
                             cfg.seq_lens, cfg.budgets, cfg.total_budget)
    return run, ref


@pytest.mark.parametrize("mode", [dict(), dict(combine=1), dict(select_mode=1), dict(select_mode=2)])
def test_prune_layer_small(csp, oracle, mode):
    cfg = _case((900, 300, 517), 4, 2, 128, 32, 32, seed=30, visual_pct=25, text_pct=50)
    if mode.get("select_mode") == 1:
        cfg.budgets = cfg.budgets[:, [0, 3]].copy()
    elif mode.get("select_mode") == 2:
        cfg.budgets = cfg.budgets.sum(axis=1, keepdims=True).astype(np.int32)
    run, ref = _run_prune(csp, oracle, cfg, **mode)
    assert run.status() == 0
    assert_scores_close(run.ss.cpu().numpy(), ref["score_self"], cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), ref["score_cross"], cfg.seq_lens, cfg.recent)
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, cfg.modality(), cfg.seq_lens,
                            cfg.recent, global_mode=mode.get("select_mode") == 1, overall=mode.get("select_mode") == 2)
    assert_selection_follows_own_scores(oracle, orc_params(oracle, cfg, **mode), run.ss.cpu().numpy(),
                                        run.sc.cpu().numpy(), run.idx.cpu().numpy(), run.n_out.cpu().numpy(),
                                        cfg.modality(), cfg.seq_lens, cfg.budgets, cfg.total_budget)
    assert_compaction_exact(run, cfg.modality())
    if not mode:
        np.testing.assert_array_equal(run.n_out.cpu().numpy(), ref["n_out"])


def test_prune_layer_without_optional_outputs_and_twice_identical(csp, oracle):
    cfg = _case((700, 450), 4, 4, 128, 32, 32, seed=31)
    run, ref = _run_prune(csp, oracle, cfg, with_optional=False)
    np.testing.assert_array_equal(run.n_out.cpu().numpy(), ref["n_out"])
    first = (run.k_out.clone(), run.v_out.clone(), run.n_out.clone())
    run.prune(with_optional=False)
    assert torch.equal(first[0], run.k_out) and torch.equal(first[1], run.v_out) and torch.equal(first[2], run.n_out)
    # compare with the run that exposes the index list
    run2, _ = _run_prune(csp, oracle, cfg)
    assert torch.equal(run2.k_out, run.k_out) and torch.equal(run2.mod_out, run.mod_out)


def test_full_budget_is_identity_and_below_total_passthrough(csp, oracle):
    cfg = _case((300, 200), 2, 2, 128, 32, 32, seed=32, visual_pct=100, text_pct=100)
    run, ref = _run_prune(csp, oracle, cfg)
    for b, L in enumerate(cfg.seq_lens):
        assert (run.n_out[b] == int(L)).all()
        np.testing.assert_array_equal(bits(run.k_out)[b, :, :L], bits(run.k)[b, :, :L])
        np.testing.assert_array_equal(bits(run.v_out)[b, :, :L], bits(run.v)[b, :, :L])
    cfg = _case((300, 200), 2, 2, 128, 32, 32, seed=33)
    cfg.total_budget = np.array([301, 100], np.int32)
    cap = 300
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    run = GpuRun(csp, gpu_params(csp, cfg, cap=cap), q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets,
                 total_budget=cfg.total_budget).prune()
    assert (run.n_out[0] == 300).all() and (run.n_out[1] < 200).all()
    np.testing.assert_array_equal(bits(run.k_out)[0, :, :300], bits(run.k)[0, :, :300])


def test_config0_full(csp, oracle):
    cfg = synth.config(0)
    run, ref = _run_prune(csp, oracle, cfg)
    assert run.status() == 0
    assert_scores_close(run.ss.cpu().numpy(), ref["score_self"], cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), ref["score_cross"], cfg.seq_lens, cfg.recent)
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, cfg.modality(), cfg.seq_lens, 16)
    assert_compaction_exact(run, cfg.modality())
    assert (run.n_out.cpu().numpy() == 520).all()


def test_config1_one_layer_full(csp, oracle):
    cfg = synth.config(1)
    run, ref = _run_prune(csp, oracle, cfg, layer=3)
    assert run.status() == 0
    assert_scores_close(run.ss.cpu().numpy(), ref["score_self"], cfg.seq_lens, cfg.recent)
    assert_scores_close(run.sc.cpu().numpy(), ref["score_cross"], cfg.seq_lens, cfg.recent)
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, cfg.modality(), cfg.seq_lens, 32)
    assert_compaction_exact(run, cfg.modality())
    assert (run.n_out.cpu().numpy() == 1027).all()


def _check_units_against_oracle(csp, oracle, cfg, run, q, k, v, units, label_row, budgets, total):
    """The oracle recomputes the listed units of a finished GPU run from the bytes the GPU read.
    units: (folded batch index fb, sequence b, KV head h).  The sampled units are laid out as a batch with one
    KV head per entry so that the oracle, which is parallel across units only, does them in one call.
    label_row(fb, b, h) -> uint8 labels of that unit, length >= L_b."""
    G, d, R = cfg.group, cfg.head_dim, cfg.recent
    n = len(units)
    all_lens = run.lens.cpu().numpy()
    lens = np.array([all_lens[fb] for fb, _, _ in units], np.int32)
    Lm, cap = int(lens.max()), run.p.out_capacity
    h_ss, h_sc, h_idx, h_n = (t.cpu().numpy() for t in (run.ss, run.sc, run.idx, run.n_out))
    qs = torch.stack([q[fb, h * G:(h + 1) * G] for fb, _, h in units]).cpu()
    ks = torch.zeros((n, 1, Lm, d), dtype=k.dtype)
    vs = torch.zeros((n, 1, Lm, d), dtype=k.dtype)
    mods = np.zeros((n, Lm), np.uint8)
    g_ss, g_sc = np.zeros((n, 1, Lm), np.float32), np.zeros((n, 1, Lm), np.float32)
    g_idx, g_n = np.full((n, 1, cap), -1, np.int32), np.zeros((n, 1), np.int32)
    for i, (fb, b, h) in enumerate(units):
        L = int(lens[i])
        ks[i, 0, :L], vs[i, 0, :L] = k[fb, h, :L].cpu(), v[fb, h, :L].cpu()
        mods[i, :L] = label_row(fb, b, h)[:L]
        g_ss[i, 0, :L], g_sc[i, 0, :L] = h_ss[fb, h, :L], h_sc[fb, h, :L]
        g_idx[i, 0], g_n[i, 0] = h_idx[fb, h], h_n[fb, h]
    bud = np.stack([budgets[b] for _, b, _ in units]).astype(np.int32)
    tot = None if total is None else np.array([total[b] for _, b, _ in units], np.int32)
    op = oracle.Params(n, G, 1, d, cfg.window, R, Lm, cap)
    ref = oracle.prune_layer(op, qs, ks, vs, mods, lens, bud, tot)
    assert_scores_close(g_ss, ref["score_self"], lens, R, "self")
    assert_scores_close(g_sc, ref["score_cross"], lens, R, "cross")
    tolerated = assert_index_sets_match(g_idx, g_n, ref, mods, lens, R)
    assert_selection_follows_own_scores(oracle, op, g_ss, g_sc, g_idx, g_n, mods, lens, bud, tot)
    return tolerated


def _expected_rows(cfg, csp):
    """Rows every head of a sequence keeps when the window is text only (disjoint supports), and whether a
    budget had to be clamped."""
    want, clamped = np.zeros(cfg.batch, np.int64), False
    for b, lay in enumerate(cfg.layouts):
        n_text, n_vis = synth.candidate_counts(lay, cfg.recent)
        ks, kc = int(cfg.budgets[b, 0]), int(cfg.budgets[b, 3])
        clamped |= ks > n_text or kc > n_vis
        want[b] = min(ks, n_text) + min(kc, n_vis) + cfg.recent
    return want, (csp.DEV_K_CLAMPED if clamped else 0)


def _full_size_check(csp, oracle, cfg, n_fold, n_sampled, first_layer=0, seed=0):
    """Full-size workload in the launch configuration the bench times: `n_fold` layers stacked on the batch
    axis of one call (n_fold = 1: one call for one layer).  Layer `first_layer` is compared in full, every
    (sequence, KV head) unit of it, and `n_sampled` seeded random (layer, sequence, KV head) units of the
    other layers are recomputed one by one.  Compaction is checked for every unit of the launch."""
    parts = [synth.make_layer(cfg, first_layer + i, "cuda") for i in range(n_fold)]
    q, k, v = (torch.cat([x[j] for x in parts], 0) for j in range(3)) if n_fold > 1 else parts[0]
    del parts
    p = gpu_params(csp, cfg)
    p.batch = cfg.batch * n_fold
    mod1 = cfg.modality()
    mod = np.tile(mod1, (n_fold, 1))
    lens = np.tile(cfg.seq_lens, n_fold)
    total = None if cfg.total_budget is None else np.tile(cfg.total_budget, n_fold)
    run = GpuRun(csp, p, q, k, v, mod, lens, np.tile(cfg.budgets, (n_fold, 1)), total_budget=total).prune()
    want, st = _expected_rows(cfg, csp)
    assert run.status() == st
    B, H = cfg.batch, cfg.n_kv_heads
    units = [(b, b, h) for b in range(B) for h in range(H)]                      # the first layer in full
    rng = np.random.RandomState(seed)
    while len(units) < B * H + n_sampled and n_fold > 1:
        layer, b, h = int(rng.randint(1, n_fold)), int(rng.randint(B)), int(rng.randint(H))
        units.append((layer * B + b, b, h))
    tolerated = 0
    for i in range(0, len(units), 256):                                          # bounded host memory per call
        tolerated += _check_units_against_oracle(csp, oracle, cfg, run, q, k, v, units[i:i + 256],
                                                 lambda fb, b, h: mod1[b], cfg.budgets, cfg.total_budget)
    assert_compaction_exact(run, mod)
    # properties that hold at any size: every layer of a sequence keeps the expected number of rows
    n = run.n_out.cpu().numpy().reshape(n_fold, B, H)
    assert (n == want[None, :, None]).all()
    return len(units), tolerated


def test_config1_all_layers_in_one_call(csp, oracle):
    n, _ = _full_size_check(csp, oracle, synth.config(1), 32, 64)
    assert n == 32 + 64


def test_config2_all_layers_in_one_call(csp, oracle):
    n, _ = _full_size_check(csp, oracle, synth.config(2), 32, 64)
    assert n == 32 + 64


def test_config3_all_layers_in_one_call(csp, oracle):
    n, _ = _full_size_check(csp, oracle, synth.config(3), 28, 64)
    assert n == 16 + 64


@pytest.mark.parametrize("budget_pct", [5, 10, 20, 40])
def test_config4_budget_sweep_round0(csp, oracle, budget_pct):
    """The serving shape is timed one call per layer over four distinct layer buffers: layer 0 in full
    (1024 units) and 64 sampled units spread over layers 1-3, at every budget of the sweep."""
    cfg = synth.config(4, budget_pct=budget_pct)
    n, _ = _full_size_check(csp, oracle, cfg, 1, 0)
    assert n == 32 * 32
    rng = np.random.RandomState(budget_pct)
    for layer in (1, 2, 3):
        q, k, v = synth.make_layer(cfg, layer, "cuda")
        mod1 = cfg.modality()
        run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod1, cfg.seq_lens, cfg.budgets,
                     total_budget=cfg.total_budget).prune()
        assert run.status() == _expected_rows(cfg, csp)[1]
        units = [(b, b, int(rng.randint(32))) for b in rng.randint(32, size=22)]
        _check_units_against_oracle(csp, oracle, cfg, run, q, k, v, units, lambda fb, b, h: mod1[b],
                                    cfg.budgets, cfg.total_budget)
        assert_compaction_exact(run, mod1)
        del run, q, k, v


@pytest.mark.parametrize("config,units", [(2, [(0, 0), (0, 17), (0, 31)]), (3, [(0, 1), (3, 2), (2, 0)])])
def test_one_layer_per_call_sampled_units(csp, oracle, config, units):
    """The other launch configuration (one call per layer: few units, large clusters)."""
    cfg = synth.config(config)
    q, k, v = synth.make_layer(cfg, 1, "cuda")
    mod1 = cfg.modality()
    run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod1, cfg.seq_lens, cfg.budgets,
                 total_budget=cfg.total_budget).prune()
    want, st = _expected_rows(cfg, csp)
    assert run.status() == st
    _check_units_against_oracle(csp, oracle, cfg, run, q, k, v, [(b, b, h) for b, h in units],
                                lambda fb, b, h: mod1[b], cfg.budgets, cfg.total_budget)
    assert_compaction_exact(run, mod1)
    assert (run.n_out.cpu().numpy() == want[:, None]).all()


def test_host_buffer_entry_point(csp, oracle):
    cfg = _case((600, 340), 4, 2, 128, 32, 32, seed=40)
    q, k, v = synth.make_layer(cfg, 0, "cpu")
    p = gpu_params(csp, cfg)
    cap = p.out_capacity
    pin = lambda t: t.contiguous().pin_memory()
    mod, lens, bud = (pin(torch.from_numpy(cfg.modality())), pin(torch.from_numpy(cfg.seq_lens)),
                      pin(torch.from_numpy(cfg.budgets)))
    k_out = pin(torch.zeros(2, 2, cap, 128, dtype=k.dtype))
    v_out = pin(torch.zeros(2, 2, cap, 128, dtype=k.dtype))
    mod_out = pin(torch.zeros(2, 2, cap, dtype=torch.uint8))
    n_out = pin(torch.zeros(2, 2, dtype=torch.int32))
    staging = torch.empty(csp.host_staging_bytes(p), dtype=torch.uint8, device="cuda")
    run = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets).prune()
    ref = oracle.prune_layer(orc_params(oracle, cfg), q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets)
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, cfg.modality(), cfg.seq_lens, cfg.recent)
    # page-locked V: its kept rows are read by the compaction kernel straight from host memory;
    # pageable V (a plain tensor): staged in full.  Same bytes either way.
    for v_host in (pin(v), v.contiguous()):
        for t in (k_out, v_out, mod_out, n_out):
            t.zero_()
        status = csp.prune_layer_host(p, pin(q), pin(k), v_host, mod, lens, bud, k_out, v_out, mod_out, n_out, staging)
        assert status == 0
        assert torch.equal(n_out, run.n_out.cpu())
        np.testing.assert_array_equal(n_out.numpy(), ref["n_out"])
        idx = run.idx.cpu().numpy()
        for b in range(2):
            for h in range(2):
                n = int(n_out[b, h])
                assert torch.equal(k_out[b, h, :n], run.k_out[b, h, :n].cpu())
                assert torch.equal(v_out[b, h, :n], run.v_out[b, h, :n].cpu())
                assert torch.equal(mod_out[b, h, :n], run.mod_out[b, h, :n].cpu())
                np.testing.assert_array_equal(bits(v_out[b, h, :n]), bits(v)[b, h][idx[b, h, :n]])
                if (idx[b, h, :n] == ref["keep_idx"][b, h, :n]).all():      # same kept set: the oracle's bytes
                    np.testing.assert_array_equal(bits(k_out[b, h, :n]), ref["k_out"][b, h, :n])
                    np.testing.assert_array_equal(bits(v_out[b, h, :n]), ref["v_out"][b, h, :n])


def test_bad_lengths_are_flagged_not_faulted(csp, oracle):
    cfg = _case((300, 200), 2, 2, 128, 32, 32, seed=41)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, cfg.modality(), [5000, -3], cfg.budgets).prune()
    assert run.status() & csp.DEV_BAD_LEN
    assert (run.n_out.cpu().numpy() == -1).all()


def test_reprune_round_with_per_head_labels(csp, oracle):
    """Second invocation of Algorithm 1: the compacted cache of round one plus appended decode
    tokens is pruned again; labels now differ per head."""
    cfg = _case((800,), 4, 2, 128, 32, 32, seed=42, visual_pct=30, text_pct=40)
    run, ref = _run_prune(csp, oracle, cfg)
    n1 = int(run.n_out[0, 0])
    assert (run.n_out == n1).all()
    add, L2 = 64, n1 + 64
    g = torch.Generator(device="cuda").manual_seed(5)
    k2 = torch.cat([run.k_out[:, :, :n1], torch.randn(1, 2, add, 128, device="cuda", generator=g).to(torch.bfloat16)], 2)
    v2 = torch.cat([run.v_out[:, :, :n1], torch.randn(1, 2, add, 128, device="cuda", generator=g).to(torch.bfloat16)], 2)
    mod2 = torch.cat([run.mod_out[:, :, :n1], torch.zeros(1, 2, add, dtype=torch.uint8, device="cuda")], 2).contiguous()
    q2 = torch.randn(1, 4, 32, 128, device="cuda", generator=g).to(torch.bfloat16)
    bud = np.array([[60, 0, 0, 20]], np.int32)
    p2 = csp.Params(1, 4, 2, 128, 32, 32, L2, 162)
    run2 = GpuRun(csp, p2, q2, k2.contiguous(), v2.contiguous(), mod2.cpu().numpy(), [L2], bud).prune()
    assert run2.status() == 0
    ref2 = oracle.prune_layer(oracle.Params(1, 4, 2, 128, 32, 32, L2, 162), q2.cpu(), k2.cpu(), v2.cpu(),
                              mod2.cpu().numpy(), np.array([L2], np.int32), bud)
    assert_scores_close(run2.ss.cpu().numpy(), ref2["score_self"], [L2], 32)
    assert_scores_close(run2.sc.cpu().numpy(), ref2["score_cross"], [L2], 32)
    assert_index_sets_match(run2.idx.cpu().numpy(), run2.n_out.cpu().numpy(), ref2, mod2.cpu().numpy(), [L2], 32)
    assert_compaction_exact(run2, mod2.cpu().numpy())


def test_reprune_rounds_in_one_buffer(csp, oracle):
    """Algorithm 1's iteration without a second cache: prune in place, append decode tokens behind the kept rows
    of the same buffer, prune in place again.  Every round is compared with a two-buffer run on the same bytes."""
    cfg = _case((800,), 4, 2, 128, 32, 32, seed=42, visual_pct=30, text_pct=40)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    p = gpu_params(csp, cfg)
    two = GpuRun(csp, p, q, k.clone(), v.clone(), cfg.modality(), cfg.seq_lens, cfg.budgets, total_budget=cfg.total_budget).prune()
    one = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets, total_budget=cfg.total_budget)
    one.k_out, one.v_out = one.k, one.v
    one.prune()
    n1 = int(two.n_out[0, 0])
    assert (two.n_out == n1).all() and torch.equal(one.n_out, two.n_out)
    assert torch.equal(one.k[:, :, :n1], two.k_out[:, :, :n1]) and torch.equal(one.v[:, :, :n1], two.v_out[:, :, :n1])
    g = torch.Generator(device="cuda").manual_seed(6)
    bud = np.array([[60, 0, 0, 20]], np.int32)
    for rnd in range(2):
        add = 64
        L2 = n1 + add
        one.k[:, :, n1:L2] = torch.randn(1, 2, add, 128, device="cuda", generator=g).to(torch.bfloat16)
        one.v[:, :, n1:L2] = torch.randn(1, 2, add, 128, device="cuda", generator=g).to(torch.bfloat16)
        mod2 = torch.cat([one.mod_out[:, :, :n1], torch.zeros(1, 2, add, dtype=torch.uint8, device="cuda")], 2)
        mod2 = torch.cat([mod2, torch.zeros(1, 2, cfg.max_len - L2, dtype=torch.uint8, device="cuda")], 2).contiguous()
        q2 = torch.randn(1, 4, 32, 128, device="cuda", generator=g).to(torch.bfloat16)
        two = GpuRun(csp, p, q2, one.k.clone(), one.v.clone(), mod2.cpu().numpy(), [L2], bud).prune()
        nxt = GpuRun(csp, p, q2, one.k, one.v, mod2.cpu().numpy(), [L2], bud)
        nxt.k_out, nxt.v_out = nxt.k, nxt.v
        nxt.prune()
        assert nxt.status() == 0 and torch.equal(nxt.n_out, two.n_out) and torch.equal(nxt.idx, two.idx)
        for h in range(2):
            n = int(two.n_out[0, h])
            assert torch.equal(nxt.k[0, h, :n], two.k_out[0, h, :n]) and torch.equal(nxt.v[0, h, :n], two.v_out[0, h, :n])
        assert torch.equal(nxt.mod_out, two.mod_out)
        if not (two.n_out == two.n_out[0, 0]).all():
            break                                         # heads diverged: a ragged append needs per-head lengths
        one, n1 = nxt, int(two.n_out[0, 0])


@pytest.mark.parametrize("budget_pct", [5, 40])
def test_config4_reprune_rounds(csp, oracle, budget_pct):
    """Batched serving shape: prune the prompt cache (round 0), then four times append 64 decode tokens to
    every head's compacted cache and prune back to the same budget (labels now differ per head).
    Sampled units are checked against the oracle in every round; structure is checked for all units."""
    cfg = synth.config(4, budget_pct=budget_pct)
    R, W, d, H = cfg.recent, cfg.window, cfg.head_dim, cfg.n_kv_heads
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    mod = cfg.modality()
    run = GpuRun(csp, gpu_params(csp, cfg), q, k, v, mod, cfg.seq_lens, cfg.budgets,
                 total_budget=cfg.total_budget).prune()
    assert run.status() & ~csp.DEV_K_CLAMPED == 0
    rng = np.random.RandomState(budget_pct)
    gen = torch.Generator(device="cuda").manual_seed(100 + budget_pct)
    totals = cfg.total_budget.astype(np.int64)
    budgets = np.array([synth.budgets_from_total(int(t), R) for t in totals], np.int32)
    for rnd in range(1, 5):
        n_prev = run.n_out.cpu().numpy()                      # [B, H] rows each head kept
        assert (n_prev > 0).all()
        lens2 = (n_prev.max(axis=1) + 64).astype(np.int32)     # heads of a sequence may differ: pad to the longest
        Lm = int(lens2.max())
        B = cfg.batch
        k2 = torch.zeros(B, H, Lm, d, dtype=torch.bfloat16, device="cuda")
        v2 = torch.zeros_like(k2)
        mod2 = torch.zeros(B, H, Lm, dtype=torch.uint8, device="cuda")
        new_k = torch.randn(B, H, 64, d, device="cuda", generator=gen).to(torch.bfloat16)
        new_v = torch.randn(B, H, 64, d, device="cuda", generator=gen).to(torch.bfloat16)
        same_len = (n_prev == n_prev[:, :1]).all()
        assert same_len, "segmented budgets with disjoint supports keep the same number of rows in every head"
        for b in range(B):
            n = int(n_prev[b, 0])
            k2[b, :, :n] = run.k_out[b, :, :n]
            v2[b, :, :n] = run.v_out[b, :, :n]
            mod2[b, :, :n] = run.mod_out[b, :, :n]
            k2[b, :, n:n + 64] = new_k[b]
            v2[b, :, n:n + 64] = new_v[b]                    # appended decode tokens are text (label 0)
        q2 = torch.randn(B, cfg.n_q_heads, W, d, device="cuda", generator=gen).to(torch.bfloat16)
        cap = int((budgets.sum(axis=1) + R).max())
        p2 = csp.Params(B, cfg.n_q_heads, H, d, W, R, Lm, cap)
        run = GpuRun(csp, p2, q2, k2, v2, mod2.cpu().numpy(), lens2, budgets, total_budget=totals.astype(np.int32))
        run.prune()
        assert run.status() & ~csp.DEV_K_CLAMPED == 0
        assert_compaction_exact(run, mod2.cpu().numpy())
        for _ in range(3):
            b, h = int(rng.randint(B)), int(rng.randint(H))
            L = int(lens2[b])
            op = oracle.Params(1, 1, 1, d, W, R, L, cap)
            ref = oracle.prune_layer(op, q2[b:b + 1, h:h + 1].cpu(), k2[b:b + 1, h:h + 1, :L].cpu(),
                                     v2[b:b + 1, h:h + 1, :L].cpu(), mod2[b:b + 1, h:h + 1, :L].cpu().numpy(),
                                     np.array([L], np.int32), budgets[b:b + 1], totals[b:b + 1].astype(np.int32))
            assert_scores_close(run.ss[b:b + 1, h:h + 1, :L].cpu().numpy(), ref["score_self"], [L], R)
            assert_scores_close(run.sc[b:b + 1, h:h + 1, :L].cpu().numpy(), ref["score_cross"], [L], R)
            assert_index_sets_match(run.idx[b:b + 1, h:h + 1].cpu().numpy(), run.n_out[b:b + 1, h:h + 1].cpu().numpy(),
                                    ref, mod2[b:b + 1, h:h + 1, :L].cpu().numpy(), [L], R)


# ------------------------------------------------------------------ a seeded sweep over shapes and modes

@pytest.mark.parametrize("seed", range(24))
def test_seeded_sweep_of_shapes_and_modes(csp, oracle, seed):
    """Random (seeded) combinations of group size, head_dim, window, recent size, batch raggedness, budgets, selection
    and combination mode, labels shared or per head, mixed-modality windows, n: the whole pass against the oracle."""
    rng = np.random.RandomState(1000 + seed)
    G = int(rng.choice([1, 1, 2, 3, 4, 7, 8]))
    n_kv = int(rng.choice([1, 2, 3]))
    d = int(rng.choice([64, 128]))
    W = int(rng.choice([1, 7, 16, 32]))
    R = int(rng.choice([0, 5, W, 40]))
    B = int(rng.randint(1, 5))
    lens = tuple(int(x) for x in rng.randint(max(W, R, 41) + 1, 1400, size=B))
    cfg = _case(lens, G * n_kv, n_kv, d, W, R, seed=seed, visual_pct=int(rng.randint(5, 90)), text_pct=int(rng.randint(5, 90)))
    mode = dict(select_mode=int(rng.choice([0, 0, 1, 2])), combine=int(rng.choice([0, 0, 1])))
    n = float(rng.choice([0.0, 1.0, 1.0, 30.0]))
    per_head = bool(rng.randint(2))
    mod = cfg.modality()
    if per_head:
        mod = np.repeat(mod[:, None, :], n_kv, axis=1).copy()
        mod[:, :, :] ^= (rng.rand(B, n_kv, cfg.max_len) < 0.1).astype(np.uint8)     # heads differ in a tenth of the labels
    if rng.randint(2):                                                              # a mixed-modality window
        for b, L in enumerate(lens):
            mod[b, ..., L - W:L] = (rng.rand(W) < 0.4).astype(np.uint8)
    nb = {0: 4, 1: 2, 2: 1}[mode["select_mode"]]
    budgets = rng.randint(0, max(2, min(lens) // 3), size=(B, nb)).astype(np.int32)
    total = rng.randint(0, 1500, size=B).astype(np.int32) if rng.randint(3) == 0 else None
    cap = int(max(lens))
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    if rng.randint(3) == 0:
        q = (q.float() * 4.0).to(cfg.dtype)                                         # peaked rows
    p = gpu_params(csp, cfg, cap=cap, n=n, **mode)
    run = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, budgets, total_budget=total).prune()
    ref = oracle.prune_layer(orc_params(oracle, cfg, cap=cap, n=n, **mode), q.cpu(), k.cpu(), v.cpu(), mod, cfg.seq_lens,
                             budgets, total)
    assert run.status() & ~csp.DEV_K_CLAMPED == 0
    assert_scores_close(run.ss.cpu().numpy(), ref["score_self"], cfg.seq_lens, R, "self")
    assert_scores_close(run.sc.cpu().numpy(), ref["score_cross"], cfg.seq_lens, R, "cross")
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, mod, cfg.seq_lens, R,
                            global_mode=mode["select_mode"] == 1, overall=mode["select_mode"] == 2)
    assert_selection_follows_own_scores(oracle, orc_params(oracle, cfg, cap=cap, n=n, **mode), run.ss.cpu().numpy(),
                                        run.sc.cpu().numpy(), run.idx.cpu().numpy(), run.n_out.cpu().numpy(), mod,
                                        cfg.seq_lens, budgets, total)
    assert_compaction_exact(run, mod)


# ------------------------------------------------------------------ many units: selection and compaction in one kernel

def _many_units_case(rng, seed, hi, n_kv, d, dtype=torch.bfloat16, G=1, min_units=300):
    """A batch with at least `min_units` (sequence, KV head) units and caches of up to `hi` positions, one of them short."""
    B = -(-min_units // n_kv) + int(rng.randint(0, 3))
    lens = [int(x) for x in rng.randint(hi // 2, hi + 1, size=B)]
    lens[0] = hi
    lens[1] = int(rng.randint(60, 200))                  # a short cache in the same call
    return _case(tuple(lens), G * n_kv, n_kv, d, 32, 32, dtype=dtype, seed=seed, visual_pct=int(rng.randint(5, 60)),
                 text_pct=int(rng.randint(5, 60)))


@pytest.mark.parametrize("seed,hi,n_kv,d,dtype,min_units", [
    (0, 2100, 16, 128, torch.bfloat16, 300), (1, 4096, 8, 128, torch.bfloat16, 300), (2, 3000, 16, 64, torch.bfloat16, 300),
    (3, 8192, 8, 64, torch.bfloat16, 300), (4, 5000, 8, 128, torch.bfloat16, 300), (5, 2500, 8, 128, torch.float32, 300),
    (6, 1100, 16, 128, torch.bfloat16, 300), (7, 2048, 8, 64, torch.bfloat16, 150), (8, 4000, 4, 128, torch.bfloat16, 150),
    (9, 1500, 8, 128, torch.float32, 200)])
def test_many_units_mid_length_caches(csp, oracle, seed, hi, n_kv, d, dtype, min_units):
    """Launches that take the fused selection + compaction kernel (at least one unit per SM, caches of 1 K - 4 K
    positions, with 4 or 8 keys per selection thread) and, beside them, some just outside that range: the whole pass
    against the oracle, and bit-identical to the three stages called one by one."""
    rng = np.random.RandomState(7000 + seed)
    cfg = _many_units_case(rng, seed, hi, n_kv, d, dtype, min_units=min_units)
    mode = dict(select_mode=int(rng.choice([0, 0, 1, 2])), combine=int(rng.choice([0, 0, 1])))
    nb = {0: 4, 1: 2, 2: 1}[mode["select_mode"]]
    B = cfg.batch
    budgets = rng.randint(0, hi // 6, size=(B, nb)).astype(np.int32)
    total = rng.randint(0, hi, size=B).astype(np.int32) if seed % 2 else None     # some caches below their budget T
    cap = int(budgets.sum(axis=1).max()) + 32 if total is None else hi
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    mod = cfg.modality()
    p = gpu_params(csp, cfg, cap=cap, **mode)
    run = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, budgets, total_budget=total).prune()
    assert run.status() & ~csp.DEV_K_CLAMPED == 0
    # the stages one by one, on the scores of the call above
    step = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, budgets, total_budget=total)
    step.ss.copy_(run.ss); step.sc.copy_(run.sc)
    step.select().compact()
    assert torch.equal(step.n_out, run.n_out)
    # and csp_select_compact on those scores, without the optional index list
    both = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, budgets, total_budget=total)
    csp.select_compact(p, run.ss, run.sc, both.k, both.v, both.mod, both.lens, both.bud, both.k_out, both.v_out,
                       both.mod_out, both.n_out, both.ws, total_budget=both.tot)
    assert both.status() & ~csp.DEV_K_CLAMPED == 0
    assert torch.equal(both.n_out, run.n_out) and torch.equal(both.k_out, run.k_out)
    assert torch.equal(both.v_out, run.v_out) and torch.equal(both.mod_out, run.mod_out)
    n_out = run.n_out.cpu().numpy()
    assert (n_out >= 0).all()
    for b in range(B):
        for h in range(n_kv):
            n = int(n_out[b, h])
            assert torch.equal(step.idx[b, h, :n], run.idx[b, h, :n])
            assert torch.equal(step.k_out[b, h, :n], run.k_out[b, h, :n])
            assert torch.equal(step.v_out[b, h, :n], run.v_out[b, h, :n])
            assert torch.equal(step.mod_out[b, h, :n], run.mod_out[b, h, :n])
            assert (run.k_out[b, h, n:] == 0).all() and (run.mod_out[b, h, n:] == 0).all()    # nothing beyond the kept rows
    assert_compaction_exact(run, mod)
    # against the oracle: a sample of sequences (all their heads), always with the longest and the short one
    pick = sorted({0, 1, *[int(x) for x in rng.choice(B, size=4, replace=False)]})
    op = oracle.Params(len(pick), cfg.n_q_heads, n_kv, d, 32, 32, cfg.max_len, cap,
                       dtype=oracle.F32 if dtype == torch.float32 else oracle.BF16, **mode)
    pad = lambda t: t[pick].cpu()
    ref = oracle.prune_layer(op, pad(q), pad(k), pad(v), mod[pick], cfg.seq_lens[pick], budgets[pick],
                             None if total is None else total[pick])
    lens = cfg.seq_lens[pick]
    assert_scores_close(run.ss[pick].cpu().numpy(), ref["score_self"], lens, 32, "self")
    assert_scores_close(run.sc[pick].cpu().numpy(), ref["score_cross"], lens, 32, "cross")
    assert_index_sets_match(run.idx[pick].cpu().numpy(), n_out[pick], ref, mod[pick], lens, 32,
                            global_mode=mode["select_mode"] == 1, overall=mode["select_mode"] == 2)
    assert_selection_follows_own_scores(oracle, op, run.ss[pick].cpu().numpy(), run.sc[pick].cpu().numpy(),
                                        run.idx[pick].cpu().numpy(), n_out[pick], mod[pick], lens, budgets[pick],
                                        None if total is None else total[pick])


def test_many_units_bad_length_and_capacity_are_flagged(csp, oracle):
    """In a launch that takes the fused kernel: a length outside [0, max_len] gives -1 rows and DEV_BAD_LEN, a unit
    whose kept rows exceed the capacity gives -1 rows and DEV_CAPACITY; the other units are unaffected; no label output."""
    rng = np.random.RandomState(7100)
    cfg = _many_units_case(rng, 9, 2600, 16, 128)
    B = cfg.batch
    budgets = np.full((B, 4), 40, np.int32)
    budgets[2] = 400                                     # 1600 + 32 rows do not fit the capacity below
    cap = 4 * 40 + 32
    lens = cfg.seq_lens.copy()
    lens[3] = cfg.max_len + 1
    lens[4] = -5
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    mod = cfg.modality()
    p = gpu_params(csp, cfg, cap=cap)
    run = GpuRun(csp, p, q, k, v, mod, lens, budgets)
    run.csp.prune_layer(p, run.q, run.k, run.v, run.mod, run.lens, run.bud, run.k_out, run.v_out, None, run.n_out,
                        run.ws, keep_idx=run.idx)
    st = run.status()
    assert st & csp.DEV_BAD_LEN and st & csp.DEV_CAPACITY and not st & csp.DEV_TIMEOUT
    n_out = run.n_out.cpu().numpy()
    assert (n_out[2] == -1).all() and (n_out[3] == -1).all() and (n_out[4] == -1).all()
    good = [b for b in range(B) if b not in (2, 3, 4)]
    assert (n_out[good] > 0).all()
    assert (run.k_out[[2, 3, 4]] == 0).all()             # nothing written for the flagged units
    assert (run.mod_out == 0).all()
    run.n_out[[2, 3, 4]] = 0
    assert_compaction_exact(run, np.zeros_like(mod))


def test_select_compact_randomized_against_the_two_calls(csp):
    """Seeded random launches inside the fused kernel's range (148-420 units, 1 K - 4 K positions, every fourth one 300 units
    or more of up to 8 K positions; head_dim, element type,
    window, recent size, selection and combination mode, shared or per-head labels, tied scores, budgets above the
    candidates, caches too short to prune, capacities that do not hold every unit): csp_select_compact must leave exactly what
    csp_select followed by csp_compact leaves, untouched rows included, and raise the same flags."""
    for it in range(60):
        rng = np.random.RandomState(50000 + it)
        H = int(rng.choice([4, 8, 16, 32]))
        B = int(rng.randint(-(-148 // H), -(-420 // H) + 1)) if it % 4 else -(-300 // H) + int(rng.randint(0, 3))
        d, dt = [(128, torch.bfloat16), (64, torch.bfloat16), (128, torch.float32), (64, torch.float32)][rng.randint(4)]
        hi = int(rng.randint(1025, 4097)) if it % 4 else int(rng.randint(4097, 8193))
        R, W = int(rng.choice([0, 7, 32, 64])), int(rng.choice([1, 16, 32]))
        lens = rng.randint(max(W, R, 2), hi + 1, size=B).astype(np.int32)
        lens[0] = hi
        if rng.randint(3) == 0:
            lens[rng.randint(B)] = int(rng.randint(0, max(W, R) + 1))
        mode, comb = int(rng.choice([0, 0, 1, 2])), int(rng.choice([0, 0, 1]))
        bud = rng.randint(0, hi // 5, size=(B, {0: 4, 1: 2, 2: 1}[mode])).astype(np.int32)
        if rng.randint(4) == 0:
            bud[rng.randint(B)] = hi
        tot = rng.randint(0, hi, size=B).astype(np.int32) if rng.randint(3) == 0 else None
        most = int(bud.sum(axis=1).max()) + R
        cap = max(1, int(rng.choice([hi, most, most - int(rng.randint(1, 50))])))
        g = torch.Generator(device="cuda")
        g.manual_seed(it)
        k = torch.randn(B, H, hi, d, device="cuda", generator=g).to(dt)
        v = torch.randn(B, H, hi, d, device="cuda", generator=g).to(dt)
        ss = torch.rand(B, H, hi, device="cuda", generator=g)
        sc = torch.rand(B, H, hi, device="cuda", generator=g)
        if rng.randint(3) == 0:
            ss, sc = (ss * 8).floor() / 8, (sc * 4).floor() / 4
        mod = (torch.rand((B, H, hi) if rng.randint(2) else (B, hi), device="cuda", generator=g) < 0.6).to(torch.uint8)
        p = csp.Params(B, H, H, d, W, R, hi, cap, dtype=csp.F32 if dt == torch.float32 else csp.BF16, select_mode=mode,
                       combine=comb)
        lens_t, bud_t = torch.from_numpy(lens).cuda(), torch.from_numpy(bud).cuda()
        tot_t = None if tot is None else torch.from_numpy(tot).cuda()
        outs = []
        for fused in (True, False):
            ko = torch.full((B, H, cap, d), 3.0, device="cuda").to(dt)
            vo = torch.full((B, H, cap, d), 5.0, device="cuda").to(dt)
            mo = torch.full((B, H, cap), 9, dtype=torch.uint8, device="cuda")
            no = torch.full((B, H), -7, dtype=torch.int32, device="cuda")
            idx = torch.full((B, H, cap), -1, dtype=torch.int32, device="cuda")
            ws = csp.new_workspace(p)
            torch.cuda.synchronize()
            if fused:
                csp.select_compact(p, ss, sc, k, v, mod, lens_t, bud_t, ko, vo, mo, no, ws, total_budget=tot_t, keep_idx=idx)
            else:
                csp.select(p, ss, sc, mod, lens_t, bud_t, idx, no, ws, total_budget=tot_t)
                csp.compact(p, k, v, mod, idx, no, ko, vo, mo)
            outs.append((ko, vo, mo, no, idx, csp.device_status(ws)))
        a, b = outs
        what = f"iteration {it}: B={B} H={H} d={d} {dt} max_len={hi} R={R} W={W} mode={mode} combine={comb} cap={cap}"
        assert a[5] == b[5] and not a[5] & csp.DEV_TIMEOUT, what
        assert torch.equal(a[3], b[3]), what
        assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) and torch.equal(a[2], b[2]), what
        kept = torch.arange(cap, device="cuda")[None, None, :] < a[3].clamp(min=0)[:, :, None]
        assert torch.equal(a[4][kept], b[4][kept]), what
