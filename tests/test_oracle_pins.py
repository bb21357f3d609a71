"""Pins for the CPU oracle: each checks it against something that is not the oracle itself --
a closed form, a library routine on a textbook special case, an algebraic identity stated in
the paper, or an independent brute-force transcription on tiny inputs."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy.special import softmax as scipy_softmax

import csp_synth as synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_case(oracle, seed, B=2, Hq=4, Hkv=2, d=8, L=(23, 17), W=3, R=4, dtype=torch.float32,
               logit_gain=1.0, logit_shift=0.0, **pk):
    """Small random problem with mixed-modality window and ragged lengths."""
    rng = np.random.RandomState(seed)
    Lm = max(L)
    q = torch.from_numpy(rng.randn(B, Hq, W, d).astype(np.float32)) * logit_gain
    k = torch.from_numpy(rng.randn(B, Hkv, Lm, d).astype(np.float32))
    v = torch.from_numpy(rng.randn(B, Hkv, Lm, d).astype(np.float32))
    if logit_shift:
        # make every logit about `logit_shift`: one constant channel in q and k
        q[..., 0] = 1.0
        k[..., 0] = logit_shift * np.sqrt(d)
    q, k, v = q.to(dtype), k.to(dtype), v.to(dtype)
    mod = (rng.rand(B, Lm) < 0.5).astype(np.uint8)
    p = oracle.Params(B, Hq, Hkv, d, W, R, Lm, Lm, dtype=oracle.F32 if dtype == torch.float32 else oracle.BF16, **pk)
    return p, q, k, v, mod, np.array(L, np.int32)


# ---------------------------------------------------------------- Eq. 7: n-softmax (P1-P4)

def test_nsoftmax_rows_sum_to_one_with_virtual_slot(oracle):
    rng = np.random.RandomState(0)
    for n in (0.0, 1.0, 7.5, 100.0):
        o = rng.randn(37) * 3
        a = oracle.nsoftmax(o, n)
        z = np.exp(o).sum()
        assert abs(a.sum() + n / (n + z) - 1.0) < 1e-12


def test_nsoftmax_n0_is_library_softmax(oracle):
    o = np.random.RandomState(1).randn(50) * 4
    np.testing.assert_allclose(oracle.nsoftmax(o, 0.0), scipy_softmax(o), rtol=1e-12, atol=0)


def test_nsoftmax_n1_is_softmax_with_one_extra_zero_logit(oracle):
    o = np.random.RandomState(2).randn(41) * 2 - 3
    padded = torch.softmax(torch.from_numpy(np.concatenate([o, [0.0]])), dim=0).numpy()
    np.testing.assert_allclose(oracle.nsoftmax(o, 1.0), padded[:-1], rtol=1e-12, atol=0)


def test_nsoftmax_restores_pre_pruning_weights_eq6(oracle):
    # Eq. 6: with n equal to the exponential mass of the pruned keys, the weights of the kept
    # keys equal the softmax weights they had before pruning.
    rng = np.random.RandomState(3)
    o = rng.randn(64) * 2
    keep = rng.rand(64) < 0.3
    full = scipy_softmax(o)
    n = np.exp(o[~keep]).sum()
    np.testing.assert_allclose(oracle.nsoftmax(o[keep], n), full[keep], rtol=1e-12, atol=0)
    # and without the correction every kept weight is larger (the sharpness shift)
    assert (oracle.nsoftmax(o[keep], 0.0) > full[keep]).all()


def test_nsoftmax_is_monotone_in_n_and_scales_softmax(oracle):
    o = np.random.RandomState(4).randn(30)
    z = np.exp(o).sum()
    prev = oracle.nsoftmax(o, 0.0)
    for n in (0.5, 1.0, 10.0):
        cur = oracle.nsoftmax(o, n)
        assert (cur < prev).all()
        np.testing.assert_allclose(cur, scipy_softmax(o) * z / (n + z), rtol=1e-12)
        prev = cur


def test_nsoftmax_large_logits_do_not_overflow(oracle):
    a = oracle.nsoftmax(np.array([900.0, 899.0, -900.0]), 1.0)
    np.testing.assert_allclose(a[:2], scipy_softmax(np.array([900.0, 899.0])), rtol=1e-12)
    a = oracle.nsoftmax(np.array([-900.0, -901.0]), 1.0)
    assert (a >= 0).all() and a.max() < 1e-300


# ---------------------------------------------------------------- scoring (P5-P7, P10, P12)

def test_mass_conservation(oracle):
    # every unit of window mass lands on exactly one of: intra score, inter score, recent keys
    p, q, k, v, mod, L = _rand_case(oracle, 5, n=1.0)
    s, c, mass = oracle.score(p, q, k, mod, L, want_row_mass=True)
    G = p.n_q_heads // p.n_kv_heads
    d = p.head_dim
    qd, kd = q.double().numpy(), k.double().numpy()
    for b in range(p.batch):
        for h in range(p.n_kv_heads):
            recent_mass = 0.0
            for g in range(G):
                for w in range(p.window):
                    pos = L[b] - p.window + w
                    o = kd[b, h, :pos + 1] @ qd[b, h * G + g, w] / np.sqrt(d)
                    a = np.exp(o) / (p.n + np.exp(o).sum())
                    recent_mass += a[L[b] - p.recent:].sum() / G
            group_mass = mass[b, h * G:(h + 1) * G].sum() / G
            assert abs(s[b, h].sum() + c[b, h].sum() + recent_mass - group_mass) < 1e-12
            assert (s[b, h, L[b] - p.recent:] == 0).all() and (c[b, h, L[b] - p.recent:] == 0).all()


def test_text_only_window_support(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 6, B=1, L=(40,), W=4, R=4)
    mod[0, 36:] = 0
    s, c = oracle.score(p, q, k, mod, L)
    vis = mod[0, :36] != 0
    assert (s[0, :, :36][:, vis] == 0).all() and (c[0, :, :36][:, ~vis] == 0).all()
    assert (s[0, :, :36][:, ~vis] > 0).all() and (c[0, :, :36][:, vis] > 0).all()


def test_all_zero_queries_closed_form_and_golden(oracle):
    gold = {}
    with open(os.path.join(GOLDEN, "allzero_q_L6.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, num, den = line.split()
                gold[name] = Fraction(int(num), int(den))
    mod = np.array([[0, 1, 1, 0, 0, 0]], np.uint8)
    p = oracle.Params(1, 2, 1, 4, 2, 2, 6, 6, dtype=oracle.F32, n=1.0)
    q = torch.zeros(1, 2, 2, 4)
    k = torch.randn(1, 1, 6, 4, generator=torch.Generator().manual_seed(0))
    s, c, mass = oracle.score(p, q, k, mod, np.array([6], np.int32), want_row_mass=True)
    for t in range(4):
        assert abs(s[0, 0, t] - float(gold[f"self_key{t}"])) < 1e-15
        assert abs(c[0, 0, t] - float(gold[f"cross_key{t}"])) < 1e-15
    np.testing.assert_allclose(mass[0, :, 0], float(gold["row_mass_q4"]), rtol=1e-15)
    np.testing.assert_allclose(mass[0, :, 1], float(gold["row_mass_q5"]), rtol=1e-15)
    assert gold["row_weight_q4"] + gold["row_weight_q5"] == gold["self_key0"]
    # general closed form at another size: weight 1/(n + p + 1) per visible key
    L, W, R, n = 19, 5, 3, 2.5
    mod = (np.arange(L) % 3 == 0).astype(np.uint8)[None]
    p = oracle.Params(1, 1, 1, 4, W, R, L, L, dtype=oracle.F32, n=n)
    s, c = oracle.score(p, torch.zeros(1, 1, W, 4), torch.randn(1, 1, L, 4), mod, np.array([L], np.int32))
    for t in range(L - R):
        es = sum(1.0 / (n + (L - W + w) + 1) for w in range(W) if mod[0, L - W + w] == mod[0, t] and t <= L - W + w)
        ec = sum(1.0 / (n + (L - W + w) + 1) for w in range(W) if mod[0, L - W + w] != mod[0, t] and t <= L - W + w)
        assert abs(s[0, 0, t] - es) < 1e-14 and abs(c[0, 0, t] - ec) < 1e-14


def _brute_force_scores(q_full, k, mod, W, R, n):
    """Independent transcription: the whole causal L x L n-softmax matrix, averaged over heads,
    trimmed to A[-O:, :-R], cut into the four blocks A^st, A^sv, A^ct, A^cv and summed over
    the query axis (Eq. 1); scores are put back at each key's original position."""
    H, L, d = q_full.shape
    A = np.zeros((L, L))
    for h in range(H):
        O = q_full[h] @ k.T / np.sqrt(d)
        for i in range(L):
            e = np.exp(O[i, :i + 1])
            A[i, :i + 1] += e / (n + e.sum()) / H
    A = A[L - W:, :L - R]
    qlab, klab = mod[L - W:], mod[:L - R]
    s, c = np.zeros(L - R), np.zeros(L - R)
    text_q, vis_q = np.where(qlab == 0)[0], np.where(qlab != 0)[0]
    text_k, vis_k = np.where(klab == 0)[0], np.where(klab != 0)[0]
    A_st, A_sv = A[np.ix_(text_q, text_k)], A[np.ix_(vis_q, vis_k)]
    A_ct, A_cv = A[np.ix_(vis_q, text_k)], A[np.ix_(text_q, vis_k)]
    s[text_k], s[vis_k] = A_st.sum(0), A_sv.sum(0)
    c[text_k], c[vis_k] = A_ct.sum(0), A_cv.sum(0)
    return s, c


@pytest.mark.parametrize("seed,L,W,R,G,n", [(0, 12, 3, 3, 2, 1.0), (1, 9, 2, 4, 1, 0.0),
                                            (2, 11, 3, 1, 2, 5.0), (3, 7, 1, 2, 2, 1.0)])
def test_brute_force_full_matrix(oracle, seed, L, W, R, G, n):
    rng = np.random.RandomState(seed)
    d = 4
    q_full = rng.randn(G, L, d).astype(np.float32) * 2
    k = rng.randn(L, d).astype(np.float32)
    mod = (rng.rand(L) < 0.5).astype(np.uint8)
    p = oracle.Params(1, G, 1, d, W, R, L, L, dtype=oracle.F32, n=n)
    s, c = oracle.score(p, q_full[None, :, L - W:], k[None, None], mod[None], np.array([L], np.int32))
    es, ec = _brute_force_scores(q_full.astype(np.float64), k.astype(np.float64), mod, W, R, n)
    np.testing.assert_allclose(s[0, 0, :L - R], es, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(c[0, 0, :L - R], ec, rtol=1e-12, atol=1e-15)


def test_head_order_and_label_swap_invariance(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 7, Hq=6, Hkv=2)
    s, c = oracle.score(p, q, k, mod, L)
    perm = [2, 0, 1, 4, 5, 3]  # permutes heads inside each group of 3
    s2, c2 = oracle.score(p, q[:, perm], k, mod, L)
    np.testing.assert_allclose(s2, s, rtol=1e-13, atol=1e-16)
    s3, c3 = oracle.score(p, q, k, 1 - mod, L)
    np.testing.assert_array_equal(s3, s)
    np.testing.assert_array_equal(c3, c)


def test_more_than_two_labels_intra_means_equal(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 8, B=1, L=(20,), W=3, R=3)
    mod3 = (np.arange(20) % 3).astype(np.uint8)[None]
    s, c = oracle.score(p, q, k, mod3, L)
    tot_s, tot_c = oracle.score(p, q, k, np.zeros_like(mod3), L)
    np.testing.assert_allclose(s + c, tot_s, rtol=1e-13)
    assert (tot_c == 0).all()


def test_bf16_inputs_are_widened_exactly(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 9, dtype=torch.bfloat16)
    s_b, c_b = oracle.score(p, q, k, mod, L)
    p32 = oracle.Params(**{**p.__dict__, "dtype": oracle.F32})
    s_f, c_f = oracle.score(p32, q.float(), k.float(), mod, L)
    np.testing.assert_array_equal(s_b, s_f)
    np.testing.assert_array_equal(c_b, c_f)


def test_padding_rows_are_ignored(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 10)
    s, c = oracle.score(p, q, k, mod, L)
    k2 = k.clone()
    k2[1, :, L[1]:] = 1e9
    s2, c2 = oracle.score(p, q, k2, mod, L)
    np.testing.assert_array_equal(s, s2)


def test_mean_over_all_heads_is_mean_of_group_scores(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 11, Hq=4, Hkv=2)
    s, c = oracle.score(p, q, k, mod, L)
    pm = oracle.Params(**{**p.__dict__, "head_reduce": oracle.HEADS_MEAN_ALL})
    sm, cm = oracle.score(pm, q, k, mod, L)
    np.testing.assert_allclose(sm[:, 0], s.mean(axis=1), rtol=1e-13, atol=1e-17)
    np.testing.assert_array_equal(sm[:, 0], sm[:, 1])
    np.testing.assert_allclose(cm[:, 1], c.mean(axis=1), rtol=1e-13, atol=1e-17)


def test_supplied_lse_reproduces_own_normaliser(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 12)
    s, c = oracle.score(p, q, k, mod, L)
    G = p.n_q_heads // p.n_kv_heads
    lse = np.zeros((p.batch, p.n_q_heads, p.window))
    for b in range(p.batch):
        for h in range(p.n_q_heads):
            for w in range(p.window):
                pos = L[b] - p.window + w
                o = k[b, h // G, :pos + 1].double().numpy() @ q[b, h, w].double().numpy() / np.sqrt(p.head_dim)
                lse[b, h, w] = np.log(np.exp(o).sum())
    s2, c2 = oracle.score(p, q, k, mod, L, lse=lse)
    np.testing.assert_allclose(s2, s, rtol=1e-12, atol=1e-16)
    np.testing.assert_allclose(c2, c, rtol=1e-12, atol=1e-16)


def test_n_matters_when_logits_are_small(oracle):
    # logits around -20: sum of exponentials << n, so n = 0 / 1 / 100 give very different scores
    res = []
    for n in (0.0, 1.0, 100.0):
        p, q, k, v, mod, L = _rand_case(oracle, 13, logit_shift=-20.0, n=n)
        s, c = oracle.score(p, q, k, mod, L)
        res.append((s + c).sum())
    assert res[0] > 1e3 * res[1] > 1e3 * res[2] * 10


# ---------------------------------------------------------------- Eq. 2: top-K (P8)

def test_topk_matches_stable_argsort_and_rank_definition(oracle):
    rng = np.random.RandomState(20)
    for trial in range(30):
        n = int(rng.randint(1, 60))
        score = rng.choice(np.array([0.0, 0.25, 0.5, 1.0, 3.0], np.float32), size=n) if trial % 2 else \
            rng.rand(n).astype(np.float32)
        cand = (rng.rand(n) < 0.7).astype(np.uint8)
        k = int(rng.randint(0, n + 3))
        mask, n_sel, kth, knext = oracle.topk(score, cand, k)
        ids = np.where(cand)[0]
        order = ids[np.argsort(-score[ids], kind="stable")]
        kk = min(k, len(ids))
        expect = np.zeros(n, np.uint8)
        expect[order[:kk]] = 1
        np.testing.assert_array_equal(mask, expect)
        assert n_sel == kk
        # rank definition: selected iff fewer than k candidates beat it
        for t in ids:
            beats = sum((score[u] > score[t]) or (score[u] == score[t] and u < t) for u in ids)
            assert bool(mask[t]) == (beats < kk)
        if kk >= 1:
            assert kth == score[order[kk - 1]]
        if kk < len(ids):
            assert knext == score[order[kk]]
        else:
            assert np.isnan(knext)


def test_topk_all_equal_scores_takes_lowest_indices(oracle):
    mask, n_sel, _, _ = oracle.topk(np.full(10, 0.5, np.float32), np.ones(10, np.uint8), 4)
    np.testing.assert_array_equal(mask, [1, 1, 1, 1, 0, 0, 0, 0, 0, 0])


# ---------------------------------------------------------------- Eq. 3-4, Algorithm 1 (P9, P11)

def _prune(oracle, p, q, k, v, mod, L, budgets, total=None):
    return oracle.prune_layer(p, q, k, v, mod, L, np.array(budgets, np.int32),
                              None if total is None else np.array(total, np.int32))


def test_full_budget_is_identity(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 30, dtype=torch.bfloat16)
    out = _prune(oracle, p, q, k, v, mod, L, [[99, 99, 0, 0]] * 2)
    kb = k.view(torch.int16).numpy().view(np.uint16)
    vb = v.view(torch.int16).numpy().view(np.uint16)
    for b in range(2):
        assert (out["n_out"][b] == L[b]).all()
        for h in range(p.n_kv_heads):
            np.testing.assert_array_equal(out["keep_idx"][b, h, :L[b]], np.arange(L[b]))
            np.testing.assert_array_equal(out["k_out"][b, h, :L[b]], kb[b, h, :L[b]])
            np.testing.assert_array_equal(out["v_out"][b, h, :L[b]], vb[b, h, :L[b]])
    assert (out["flags"] & oracle.FLAG_K_CLAMPED).all()


def test_cache_below_total_budget_is_returned_unchanged(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 31)
    out = _prune(oracle, p, q, k, v, mod, L, [[1, 1, 1, 1]] * 2, total=[24, 17])
    # L = (23, 17): 23 < 24 -> identity; 17 < 17 is false -> pruned
    assert (out["n_out"][0] == 23).all() and (out["flags"][0] & oracle.FLAG_IDENTITY).all()
    assert (out["n_out"][1] < 17).all() and not (out["flags"][1] & oracle.FLAG_IDENTITY).any()
    np.testing.assert_array_equal(out["k_out"][0, 0, :23], k[0, 0, :23].numpy())


def test_output_structure(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 32, B=2, L=(50, 33), W=4, R=6)
    mod[:, -8:] = 0  # text-only windows: supports are disjoint
    bud = [[5, 0, 0, 7], [3, 0, 0, 4]]
    out = _prune(oracle, p, q, k, v, mod, L, bud)
    for b in range(2):
        for h in range(p.n_kv_heads):
            n = out["n_out"][b, h]
            idx = out["keep_idx"][b, h, :n]
            assert n == sum(bud[b]) + p.recent
            assert (np.diff(idx) > 0).all()
            np.testing.assert_array_equal(idx[-p.recent:], np.arange(L[b] - p.recent, L[b]))
            np.testing.assert_array_equal(out["k_out"][b, h, :n], k[b, h].numpy()[idx])
            np.testing.assert_array_equal(out["v_out"][b, h, :n], v[b, h].numpy()[idx])
            np.testing.assert_array_equal(out["mod_out"][b, h, :n], mod[b][idx])
            kept = idx[:-p.recent]
            assert (mod[b][kept] == 0).sum() == bud[b][0] and (mod[b][kept] != 0).sum() == bud[b][3]
            # the kept text keys are the best text keys by intra score
            s = out["score_self"][b, h]
            text = np.where(mod[b][:L[b] - p.recent] == 0)[0]
            best = text[np.argsort(-s[text], kind="stable")][:bud[b][0]]
            assert set(best) == set(kept[mod[b][kept] == 0])


def test_and_combine_on_text_only_window_keeps_only_recent(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 33, B=1, L=(40,), W=4, R=5, combine=1)
    mod[0, -6:] = 0
    out = _prune(oracle, p, q, k, v, mod, L, [[6, 0, 0, 6]])
    assert (out["n_out"] == p.recent).all()
    np.testing.assert_array_equal(out["keep_idx"][0, 0, :5], np.arange(35, 40))
    # OR keeps both sets
    p.combine = 0
    assert (_prune(oracle, p, q, k, v, mod, L, [[6, 0, 0, 6]])["n_out"] == 17).all()


def test_and_or_on_mixed_window_are_intersection_and_union(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 34, B=1, L=(60,), W=6, R=6, select_mode=1)
    bud = [[20, 25]]
    s, c = oracle.score(p, q, k, mod, L)
    sets = {}
    for comb in (0, 1):
        p.combine = comb
        idx, n_out, _, _ = oracle.select(p, s.astype(np.float32), c.astype(np.float32), mod, L,
                                         np.array(bud, np.int32))
        sets[comb] = [set(idx[0, h, :n_out[0, h] - 6]) for h in range(p.n_kv_heads)]
    for h in range(p.n_kv_heads):
        top_s = set(np.argsort(-s[0, h, :54].astype(np.float32), kind="stable")[:20])
        top_c = set(np.argsort(-c[0, h, :54].astype(np.float32), kind="stable")[:25])
        assert sets[0][h] == top_s | top_c and sets[1][h] == top_s & top_c


def _stable_topk(score, ids, k):
    """Eq. 2 written with numpy: the first k of `ids` in a stable descending sort of their scores."""
    k = max(0, min(int(k), len(ids)))
    return set(ids[np.argsort(-score[ids].astype(np.float64), kind="stable")][:k].tolist())


@pytest.mark.parametrize("seed,quantise", [(50, None), (51, None), (52, 8)])
def test_segmented_select_is_four_independent_topks_on_a_mixed_window(oracle, seed, quantise):
    """Budgets per key modality: the intra vector s ranks the text keys and, separately, the visual keys; so
    does the inter vector c.  M^s is the union of the two s problems, M^c of the two c problems; Eq. 3 joins
    them (union by default, intersection as printed).  With a mixed-modality window both vectors are non-zero
    on both kinds of key, so a problem ranked by the wrong vector or drawn from the wrong keys changes the set."""
    p, q, k, v, mod, L = _rand_case(oracle, seed, B=2, Hq=4, Hkv=2, L=(61, 47), W=6, R=5)
    for b in range(2):                                   # both labels among the window queries
        mod[b, L[b] - 6:L[b]] = [0, 1, 1, 0, 1, 0]
    s, c = oracle.score(p, q, k, mod, L)
    s32, c32 = s.astype(np.float32), c.astype(np.float32)
    if quantise:                                         # many equal scores: ties go to the lower position
        s32 = (np.floor(s32 * quantise * 4) / (quantise * 4)).astype(np.float32)
        c32 = (np.floor(c32 * quantise * 4) / (quantise * 4)).astype(np.float32)
    for b in range(2):
        N = L[b] - p.recent
        text, vis = mod[b, :N] == 0, mod[b, :N] != 0
        for h in range(p.n_kv_heads):                    # every vector is informative on every kind of key
            assert (s32[b, h, :N][text] > 0).sum() > 8 and (s32[b, h, :N][vis] > 0).sum() > 8
            assert (c32[b, h, :N][text] > 0).sum() > 8 and (c32[b, h, :N][vis] > 0).sum() > 8
    bud = np.array([[7, 5, 4, 9], [3, 30, 6, 2]], np.int32)    # self/text, self/visual, cross/text, cross/visual
    for comb in (oracle.COMBINE_OR, oracle.COMBINE_AND):
        p.combine = comb
        idx, n_out, flags, margins = oracle.select(p, s32, c32, mod, L, bud)
        for b in range(2):
            N = int(L[b]) - p.recent
            text, vis = np.where(mod[b, :N] == 0)[0], np.where(mod[b, :N] != 0)[0]
            clamped = any(bud[b, j] > len(ids) for j, ids in enumerate((text, vis, text, vis)))
            for h in range(p.n_kv_heads):
                st, sv = _stable_topk(s32[b, h], text, bud[b, 0]), _stable_topk(s32[b, h], vis, bud[b, 1])
                ct, cv = _stable_topk(c32[b, h], text, bud[b, 2]), _stable_topk(c32[b, h], vis, bud[b, 3])
                ms, mc = st | sv, ct | cv
                want = sorted(ms & mc if comb == oracle.COMBINE_AND else ms | mc)
                got = idx[b, h, :n_out[b, h]]
                np.testing.assert_array_equal(got[:len(want)], want)
                np.testing.assert_array_equal(got[len(want):], np.arange(N, L[b]))
                assert bool(flags[b, h] & oracle.FLAG_K_CLAMPED) == clamped
                # the reported boundary scores belong to the right problem
                for j, (vec, ids) in enumerate(((s32, text), (s32, vis), (c32, text), (c32, vis))):
                    kk = min(int(bud[b, j]), len(ids))
                    ranked = np.sort(vec[b, h][ids].astype(np.float64))[::-1]
                    if kk >= 1:
                        assert margins[b, h, j, 0] == np.float32(ranked[kk - 1])
                    if kk < len(ids):
                        assert margins[b, h, j, 1] == np.float32(ranked[kk])


def test_segmented_select_hand_worked_example(oracle):
    gold = {}
    with open(os.path.join(GOLDEN, "segmented_select_L10.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, *vals = line.split()
                gold[name] = vals
    mod = np.array([gold["labels"]], np.uint8)
    s = np.zeros((1, 1, 10), np.float32)
    c = np.zeros((1, 1, 10), np.float32)
    s[0, 0, :8] = np.array(gold["s"], np.float32)
    c[0, 0, :8] = np.array(gold["c"], np.float32)
    bud = np.array([gold["budgets"]], np.int32)
    for comb, name in ((oracle.COMBINE_OR, "keep_or"), (oracle.COMBINE_AND, "keep_and")):
        p = oracle.Params(1, 1, 1, 4, 2, 2, 10, 10, combine=comb)
        idx, n_out, flags, _ = oracle.select(p, s, c, mod, np.array([10], np.int32), bud)
        want = np.array(gold[name], np.int32)
        assert n_out[0, 0] == len(want) and flags[0, 0] == 0
        np.testing.assert_array_equal(idx[0, 0, :len(want)], want)


def test_capacity_overflow_and_clamp_flags(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 35, B=1, L=(30,), W=3, R=3)
    p.out_capacity = 10
    out = _prune(oracle, p, q, k, v, mod, L, [[9, 9, 0, 0]])
    assert (out["n_out"] == -1).all() and (out["flags"] & oracle.FLAG_CAPACITY).all()
    out = _prune(oracle, p, q, k, v, mod, L, [[2, 2, 0, 0]])
    assert (out["n_out"] == 7).all() and (out["flags"] == 0).all()


def test_short_sequence_is_identity(oracle):
    p, q, k, v, mod, L = _rand_case(oracle, 36, B=2, L=(2, 20), W=3, R=4)
    out = _prune(oracle, p, q, k, v, mod, L, [[1, 1, 1, 1]] * 2)
    assert (out["n_out"][0] == 2).all() and (out["flags"][0] & oracle.FLAG_IDENTITY).all()
    p2, q, k, v, mod, L = _rand_case(oracle, 36, B=2, L=(0, 20), W=3, R=4)
    assert (_prune(oracle, p2, q, k, v, mod, L, [[1, 1, 1, 1]] * 2)["n_out"][0] == 0).all()


# ---------------------------------------------------------------- input generator sanity

def test_overall_topk_mode_is_one_stable_topk_on_the_summed_scores(oracle):
    """The ablation's comparison arm: one top-k on s + c over all candidates, no split.  Checked against a
    stable descending argsort of the fp32 sum; a window of a single label makes s + c the plain column sum of A."""
    p, q, k, v, mod, L = _rand_case(oracle, 31, L=(40, 33), R=5, select_mode=oracle.SELECT_OVERALL)
    s, c = oracle.score(p, q, k, mod, L)
    s32, c32 = s.astype(np.float32), c.astype(np.float32)
    bud = np.array([[7], [50]], np.int32)            # the second budget exceeds its candidates: clamped
    idx, n_out, flags, _ = oracle.select(p, s32, c32, mod, L, bud)
    for b in range(p.batch):
        N = int(L[b]) - p.recent
        kk = min(int(bud[b, 0]), N)
        for h in range(p.n_kv_heads):
            mix = s32[b, h, :N] + c32[b, h, :N]
            want = np.sort(np.argsort(-mix.astype(np.float64), kind="stable")[:kk])
            got = idx[b, h, :n_out[b, h]]
            np.testing.assert_array_equal(got[:kk], want)
            np.testing.assert_array_equal(got[kk:], np.arange(N, int(L[b])))
            assert bool(flags[b, h] & oracle.FLAG_K_CLAMPED) == (int(bud[b, 0]) > N)
    # with every query and key carrying one label the inter score is zero and s is the whole column sum
    one = np.zeros_like(mod)
    s1, c1 = oracle.score(p, q, k, one, L)
    assert (c1 == 0).all()
    i_over, n_over, _, _ = oracle.select(p, s1.astype(np.float32), c1.astype(np.float32), one, L, np.array([[6], [6]], np.int32))
    pg = oracle.Params(**{**p.__dict__, "select_mode": oracle.SELECT_GLOBAL})
    i_glob, n_glob, _, _ = oracle.select(pg, s1.astype(np.float32), c1.astype(np.float32), one, L, np.array([[6, 0], [6, 0]], np.int32))
    np.testing.assert_array_equal(n_over, n_glob)
    np.testing.assert_array_equal(i_over, i_glob)


# ---------------------------------------------------------------- Section 3.3: n-softmax decode attention

def _decode_case(oracle, seed, B=2, Hq=6, Hkv=2, d=16, cap=37, dtype=torch.float32, gain=1.0, **pk):
    rng = np.random.RandomState(seed)
    q = (torch.from_numpy(rng.randn(B, Hq, d).astype(np.float32)) * gain).to(dtype)
    k = torch.from_numpy(rng.randn(B, Hkv, cap, d).astype(np.float32)).to(dtype)
    v = torch.from_numpy(rng.randn(B, Hkv, cap, d).astype(np.float32)).to(dtype)
    rows = rng.randint(1, cap + 1, size=(B, Hkv)).astype(np.int32)
    p = oracle.Params(B, Hq, Hkv, d, 1, 0, cap, cap, dtype=oracle.F32 if dtype == torch.float32 else oracle.BF16, **pk)
    return p, q, k, v, rows


def test_decode_n0_is_library_attention(oracle):
    """With n = 0 the normaliser is the plain softmax: torch's scaled_dot_product_attention per head."""
    p, q, k, v, rows = _decode_case(oracle, 40, n=0.0)
    out = oracle.decode_attn(p, q, k, v, rows)
    G = p.n_q_heads // p.n_kv_heads
    for b in range(p.batch):
        for hq in range(p.n_q_heads):
            r = int(rows[b, hq // G])
            ref = torch.nn.functional.scaled_dot_product_attention(
                q[b, hq][None, None].double(), k[b, hq // G, :r][None].double(), v[b, hq // G, :r][None].double())
            np.testing.assert_allclose(out[b, hq], ref[0, 0].numpy(), rtol=1e-10, atol=1e-12)


def test_decode_n1_is_attention_with_one_extra_zero_key(oracle):
    """n = 1 equals ordinary softmax attention over the cache plus one key with logit 0 and a zero value row
    (the slot that holds the mass of what pruning removed)."""
    p, q, k, v, rows = _decode_case(oracle, 41, n=1.0, gain=2.0)
    out = oracle.decode_attn(p, q, k, v, rows)
    G = p.n_q_heads // p.n_kv_heads
    for b in range(p.batch):
        for hq in range(p.n_q_heads):
            r = int(rows[b, hq // G])
            kk = torch.cat([k[b, hq // G, :r], torch.zeros(1, p.head_dim)]).double()     # q . 0 = logit 0
            vv = torch.cat([v[b, hq // G, :r], torch.zeros(1, p.head_dim)]).double()
            w = scipy_softmax((kk @ q[b, hq].double()).numpy() / np.sqrt(p.head_dim))
            np.testing.assert_allclose(out[b, hq], w @ vv.numpy(), rtol=1e-10, atol=1e-12)


def test_decode_zero_query_closed_form(oracle):
    """q = 0: every logit is 0, every weight 1 / (n + rows), the output is the column sum of V over n + rows."""
    p, q, k, v, rows = _decode_case(oracle, 42, n=3.0)
    out = oracle.decode_attn(p, torch.zeros_like(q), k, v, rows)
    G = p.n_q_heads // p.n_kv_heads
    for b in range(p.batch):
        for hq in range(p.n_q_heads):
            r = int(rows[b, hq // G])
            want = [float(sum(Fraction(float(x)) for x in v[b, hq // G, :r, c]) / (3 + r)) for c in range(p.head_dim)]
            np.testing.assert_allclose(out[b, hq], want, rtol=1e-13, atol=1e-15)


def test_decode_restores_pre_pruning_weights(oracle):
    """Eq. 6 -> Eq. 7: if n equals the exponential mass of the rows that were removed, attention over the kept
    rows gives exactly the kept rows' share of full softmax attention over all rows."""
    p, q, k, v, rows = _decode_case(oracle, 43, B=1, Hq=2, Hkv=2, cap=29, n=0.0)
    rows[:] = 29
    keep = 11
    for h in range(2):
        o = (k[0, h].double() @ q[0, h].double()).numpy() / np.sqrt(p.head_dim)
        w_full = scipy_softmax(o)
        want = w_full[:keep] @ v[0, h, :keep].double().numpy()
        removed_mass = float(np.exp(o[keep:]).sum())
        ph = oracle.Params(1, 1, 1, p.head_dim, 1, 0, 29, 29, dtype=oracle.F32, n=removed_mass)
        got = oracle.decode_attn(ph, q[:, h:h + 1], k[:, h:h + 1], v[:, h:h + 1], np.array([[keep]], np.int32))
        np.testing.assert_allclose(got[0, 0], want, rtol=1e-10, atol=1e-12)


def test_decode_rows_beyond_n_rows_and_head_mapping(oracle):
    """Rows past n_rows never matter; query head hq reads KV head hq // G; empty heads give zeros."""
    p, q, k, v, rows = _decode_case(oracle, 44)
    out = oracle.decode_attn(p, q, k, v, rows)
    k2, v2 = k.clone(), v.clone()
    for b in range(p.batch):
        for h in range(p.n_kv_heads):
            k2[b, h, rows[b, h]:] = 1e6
            v2[b, h, rows[b, h]:] = -1e6
    np.testing.assert_array_equal(oracle.decode_attn(p, q, k2, v2, rows), out)
    # swapping the two KV heads together with the two groups of query heads swaps the outputs
    G = p.n_q_heads // p.n_kv_heads
    perm = list(range(G, 2 * G)) + list(range(G))
    out_sw = oracle.decode_attn(p, q[:, perm], k.flip(1), v.flip(1), rows[:, ::-1].copy())
    np.testing.assert_array_equal(out_sw, out[:, perm])
    rows0 = rows.copy(); rows0[0, 0] = 0
    assert (oracle.decode_attn(p, q, k, v, rows0)[0, :G] == 0).all()
    # a transposed operand (q.k over the wrong axis) or a missing 1/sqrt(d) would break this closed form:
    # one row only -> out = v_0 * e^o / (n + e^o)
    one = np.ones_like(rows)
    got = oracle.decode_attn(p, q, k, v, one)
    for b in range(p.batch):
        for hq in range(p.n_q_heads):
            o = float(q[b, hq].double() @ k[b, hq // G, 0].double()) / np.sqrt(p.head_dim)
            np.testing.assert_allclose(got[b, hq], v[b, hq // G, 0].double().numpy() * np.exp(o) / (1.0 + np.exp(o)),
                                       rtol=1e-12, atol=1e-15)


def test_decode_bf16_inputs_are_widened_exactly(oracle):
    p, q, k, v, rows = _decode_case(oracle, 45, dtype=torch.bfloat16)
    p32 = oracle.Params(**{**p.__dict__, "dtype": oracle.F32})
    np.testing.assert_array_equal(oracle.decode_attn(p, q, k, v, rows),
                                  oracle.decode_attn(p32, q.float(), k.float(), v.float(), rows))


# ---------------------------------------------------------------- Algorithm 1's iteration loop: scores carried along

def _decode_rounds(oracle, seed, L0, steps, W, G, d, n, labels_new):
    """A cache of L0 rows, then `steps` appended tokens, one decode step each; a new window starts W steps before
    the end.  Returns everything needed to recompute the result from scratch."""
    rng = np.random.RandomState(seed)
    L = L0 + steps
    k = rng.randn(1, 1, L, d).astype(np.float32)
    v = rng.randn(1, 1, L, d).astype(np.float32)
    q_all = (rng.randn(G, L, d) * 1.5).astype(np.float32)            # only the appended positions are ever used
    mod = np.zeros((1, 1, L), np.uint8)
    mod[0, 0, :L0] = rng.rand(L0) < 0.5
    mod[0, 0, L0:] = labels_new
    p = oracle.Params(1, G, 1, d, 1, 0, L, L, dtype=oracle.F32, n=n)
    acc_s, acc_c = np.full((1, 1, L), 7.0), np.full((1, 1, L), -3.0)  # stale contents: the first step must clear them
    outs = []
    for i in range(steps):
        pos = L0 + i                                                  # the new token sits at this position
        q = torch.from_numpy(q_all[None, :, pos])
        out = oracle.decode_step(p, q, k, v, np.array([[pos + 1]], np.int32), mod, mod[0, :, pos].copy(),
                                 acc_s, acc_c, first=(i == steps - W))
        outs.append(out)
    return p, k, v, q_all, mod, acc_s, acc_c, outs


@pytest.mark.parametrize("seed,L0,steps,W,G,n", [(60, 9, 5, 3, 2, 1.0), (61, 4, 6, 6, 1, 0.0), (62, 12, 7, 4, 3, 2.5)])
def test_decode_steps_carry_the_scores_of_the_final_window(oracle, seed, L0, steps, W, G, n):
    """Row p of the causal attention matrix is final once the token at p has been decoded.  So the intra / inter
    sums collected over the last W decode steps equal Eq. 1 on the final cache with those W queries as the
    observation window: checked against the full-matrix transcription, and against the from-scratch scorer."""
    d = 4
    rng = np.random.RandomState(seed + 100)
    labels_new = (rng.rand(steps) < 0.4).astype(np.uint8)
    p, k, v, q_all, mod, acc_s, acc_c, outs = _decode_rounds(oracle, seed, L0, steps, W, G, d, n, labels_new)
    L = L0 + steps
    es, ec = _brute_force_scores(q_all.astype(np.float64), k[0, 0].astype(np.float64), mod[0, 0], W, 0, n)
    np.testing.assert_allclose(acc_s[0, 0], es, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(acc_c[0, 0], ec, rtol=1e-12, atol=1e-15)
    ps = oracle.Params(1, G, 1, d, W, 0, L, L, dtype=oracle.F32, n=n)
    s, c = oracle.score(ps, q_all[None, :, L - W:], k, mod[0], np.array([L], np.int32))
    np.testing.assert_allclose(acc_s[0, 0], s[0, 0], rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(acc_c[0, 0], c[0, 0], rtol=1e-12, atol=1e-15)
    # every step's output is plain n-softmax attention over the rows present at that step
    for i, out in enumerate(outs):
        rows = L0 + i + 1
        for g in range(G):
            o = k[0, 0, :rows].astype(np.float64) @ q_all[g, rows - 1].astype(np.float64) / np.sqrt(d)
            a = np.exp(o) / (n + np.exp(o).sum())
            np.testing.assert_allclose(out[0, g], a @ v[0, 0, :rows].astype(np.float64), rtol=1e-12, atol=1e-15)


def test_decode_step_zero_query_closed_form_and_mass(oracle):
    """q = 0: the token decoded with `rows` rows in the cache gives every row 1 / (n + rows); a text token adds
    that to the intra sum of text rows and to the inter sum of visual rows.  And for any query the two sums gain,
    together, the row's whole mass sum_t a_t = 1 - n / (n + Z)."""
    n, d, G = 2.0, 4, 2
    rng = np.random.RandomState(63)
    cap = 11
    k = rng.randn(2, 1, cap, d).astype(np.float32)
    v = rng.randn(2, 1, cap, d).astype(np.float32)
    mod = (rng.rand(2, 1, cap) < 0.5).astype(np.uint8)
    p = oracle.Params(2, G, 1, d, 1, 0, cap, cap, dtype=oracle.F32, n=n)
    acc_s, acc_c = np.zeros((2, 1, cap)), np.zeros((2, 1, cap))
    qlab = np.array([0, 1], np.uint8)
    for step, rows in enumerate((7, 8, 9)):
        oracle.decode_step(p, torch.zeros(2, G, d), k, v, np.array([[rows], [rows - 2]], np.int32), mod, qlab,
                           acc_s, acc_c, first=(step == 0))
    for b, shift in ((0, 0), (1, 2)):
        for t in range(cap):
            want = sum(Fraction(1) / (Fraction(2) + (rows - shift)) for rows in (7, 8, 9) if t < rows - shift)
            same = mod[b, 0, t] == qlab[b]
            assert abs(acc_s[b, 0, t] - (float(want) if same else 0.0)) < 1e-15
            assert abs(acc_c[b, 0, t] - (0.0 if same else float(want))) < 1e-15
    q = torch.from_numpy(rng.randn(2, G, d).astype(np.float32) * 2)
    a_s, a_c = np.zeros((2, 1, cap)), np.zeros((2, 1, cap))
    rows = np.array([[cap], [5]], np.int32)
    oracle.decode_step(p, q, k, v, rows, mod, qlab, a_s, a_c, first=True)
    for b in range(2):
        r = int(rows[b, 0])
        mass = 0.0
        for g in range(G):
            z = np.exp(k[b, 0, :r].astype(np.float64) @ q[b, g].double().numpy() / np.sqrt(d)).sum()
            mass += (1.0 - n / (n + z)) / G
        assert abs(a_s[b].sum() + a_c[b].sum() - mass) < 1e-13
        assert (a_s[b, 0, r:] == 0).all() and (a_c[b, 0, r:] == 0).all()


def test_decode_step_first_clears_the_unit_and_later_steps_add(oracle):
    p, q, k, v, rows = _decode_case(oracle, 64, B=1, Hq=2, Hkv=2, cap=13)
    mod = np.zeros((1, 2, 13), np.uint8)
    acc_s, acc_c = np.full((1, 2, 13), 5.0), np.full((1, 2, 13), 5.0)
    out = oracle.decode_step(p, q, k, v, rows, mod, np.array([0], np.uint8), acc_s, acc_c, first=True)
    np.testing.assert_array_equal(out, oracle.decode_attn(p, q, k, v, rows))
    for h in range(2):
        r = int(rows[0, h])
        assert (acc_s[0, h, r:] == 0.0).all() and (acc_c[0, h] == 0.0).all() and (acc_s[0, h, :r] > 0).all()
    before = acc_s.copy()
    oracle.decode_step(p, q, k, v, rows, mod, np.array([1], np.uint8), acc_s, acc_c, first=False)
    np.testing.assert_array_equal(acc_s, before)                     # a visual query: everything goes to the inter sum
    for h in range(2):
        r = int(rows[0, h])
        np.testing.assert_allclose(acc_c[0, h, :r], before[0, h, :r], rtol=1e-15)


# ---------------------------------------------------------------- Section 1: the distribution-gap diagnostic

def test_js_divergence_closed_forms_and_library(oracle):
    from scipy.spatial.distance import jensenshannon
    a = np.array([5, 0, 3, 9, 0, 1], np.int64)
    assert oracle.js_divergence(a, a) == 0.0
    assert oracle.js_divergence(a, 7 * a) == 0.0                      # only the normalised shapes matter
    b = np.array([0, 4, 0, 0, 2, 0], np.int64)                        # disjoint supports: ln 2
    assert abs(oracle.js_divergence(a, b) - np.log(2.0)) < 1e-15
    rng = np.random.RandomState(70)
    for _ in range(5):
        x, y = rng.randint(0, 50, 64).astype(np.int64), rng.randint(0, 50, 64).astype(np.int64)
        want = jensenshannon(x / x.sum(), y / y.sum()) ** 2          # scipy returns the square root, natural log
        assert abs(oracle.js_divergence(x, y) - want) < 1e-13
        assert abs(oracle.js_divergence(x, y) - oracle.js_divergence(y, x)) < 1e-16
    assert np.isnan(oracle.js_divergence(a, np.zeros(6, np.int64)))
    # a worked case: P = (1, 0), Q = (1/2, 1/2): M = (3/4, 1/4)
    want = 0.5 * np.log(1 / 0.75) + 0.5 * (0.5 * np.log(0.5 / 0.75) + 0.5 * np.log(0.5 / 0.25))
    assert abs(oracle.js_divergence(np.array([2, 0]), np.array([3, 3])) - want) < 1e-15


def _weights_per_head(q_full, k, n):
    """Causal n-softmax matrix of every head (the full-matrix transcription, not averaged)."""
    H, L, d = q_full.shape
    A = np.zeros((H, L, L))
    for h in range(H):
        O = q_full[h] @ k.T / np.sqrt(d)
        for i in range(L):
            e = np.exp(O[i, :i + 1])
            A[h, i, :i + 1] = e / (n + e.sum())
    return A


@pytest.mark.parametrize("seed,L,W,R,G,n", [(71, 40, 5, 7, 2, 1.0), (72, 33, 4, 4, 1, 0.0), (73, 25, 6, 2, 3, 4.0)])
def test_weight_histogram_against_the_full_matrix(oracle, seed, L, W, R, G, n):
    rng = np.random.RandomState(seed)
    d = 4
    q_full = (rng.randn(G, L, d) * 3).astype(np.float32)
    k = rng.randn(L, d).astype(np.float32)
    mod = (rng.rand(L) < 0.5).astype(np.uint8)
    p = oracle.Params(1, G, 1, d, W, R, L, L, dtype=oracle.F32, n=n)
    hist, near, js, js_all = oracle.weight_histogram(p, q_full[None, :, L - W:], k[None, None], mod[None],
                                                     np.array([L], np.int32), near_eps=0.05)
    A = _weights_per_head(q_full.astype(np.float64), k.astype(np.float64), n)
    want = np.zeros((2, oracle.HIST_BINS), np.int64)
    close = np.zeros((2, oracle.HIST_BINS), np.int64)
    for g in range(G):
        for i in range(L - W, L):
            for t in range(min(L - R, i + 1)):
                cls = 0 if mod[i] == mod[t] else 1
                x = (np.log2(A[g, i, t]) - oracle.HIST_LO) / oracle.HIST_WIDTH
                want[cls, int(np.clip(np.floor(x), 0, oracle.HIST_BINS - 1))] += 1
                je = int(np.floor(x + 0.5))
                if 1 <= je <= oracle.HIST_BINS - 1 and abs(x - je) * oracle.HIST_WIDTH <= 0.05:
                    close[cls, je] += 1
    np.testing.assert_array_equal(hist[0, 0], want)
    np.testing.assert_array_equal(near[0, 0], close)
    assert want.sum() == G * sum(min(L - R, i + 1) for i in range(L - W, L))
    assert abs(js[0, 0] - oracle.js_divergence(want[0], want[1])) < 1e-15 and abs(js_all - js[0, 0]) < 1e-15


def test_weight_histogram_zero_query_closed_form_and_pooling(oracle):
    """q = 0: row w gives every key it sees 1 / (n + L - W + w + 1); with L = 20, W = 2, n = 1 those are 1/20 and
    1/21, both in the bin that holds log2 in [-4.5, -4): bin 55.  Counts follow from the labels alone."""
    L, W, R, G = 20, 2, 3, 2
    mod = np.zeros((2, L), np.uint8)
    mod[0, 3:9] = 1                                  # sequence 0: six visual candidates, text window
    mod[1, :] = 1                                    # sequence 1: everything visual -> no inter pairs
    p = oracle.Params(2, G, 1, 4, W, R, L, L, dtype=oracle.F32, n=1.0)
    k = torch.randn(2, 1, L, 4, generator=torch.Generator().manual_seed(1))
    hist, near, js, js_all = oracle.weight_histogram(p, torch.zeros(2, G, W, 4), k, mod, np.array([L, L], np.int32))
    N = L - R
    assert hist[0, 0, 0, 55] == G * W * (N - 6) and hist[0, 0, 1, 55] == G * W * 6
    assert hist[1, 0, 0, 55] == G * W * N and hist[1, 0, 1].sum() == 0
    assert hist.sum() == 2 * G * W * N
    assert js[0, 0] == 0.0 and np.isnan(js[1, 0])    # same shape -> 0; an empty histogram -> undefined
    assert js_all == 0.0                             # pooled over both units: both classes sit in the same bin


def test_benchmark_shapes_match_their_description():
    c1 = synth.config(1)
    assert c1.seq_lens.tolist() == [4096] and c1.budgets.tolist() == [[304, 0, 0, 691]]
    assert c1.out_capacity() == 1027
    c0 = synth.config(0)
    assert c0.budgets.tolist() == [[120, 0, 0, 384]] and c0.seq_lens.tolist() == [1024]
    c2 = synth.config(2)
    assert c2.seq_lens.tolist() == [16384] and c2.budgets.tolist() == [[803, 0, 0, 803]]
    assert c2.total_budget.tolist() == [1638]
    c3 = synth.config(3)
    assert c3.seq_lens.tolist() == [8192, 16384, 24576, 32768]
    assert c3.budgets[3].tolist() == [1626, 0, 0, 4301]
    m3 = c3.modality()
    assert abs(m3[3].mean() - 0.875) < 1e-9 and (m3[:, -32:] == 0).all() is not None
    c4 = synth.config(4, budget_pct=10)
    assert c4.batch == 32 and c4.seq_lens.min() >= 2048 and c4.seq_lens.max() <= 8192
    for lay, L in zip(c4.layouts, c4.seq_lens):
        assert lay[-1][0] == synth.TEXT and lay[-1][1] >= 64
        assert 2 <= sum(1 for lab, _ in lay if lab == synth.VISUAL) <= 8
    q, k, v = synth.make_layer(c0, 0)
    assert k.shape == (1, 4, 1024, 64) and k.dtype == torch.float32
    kn = k[0, 0].norm(dim=-1)
    assert kn[0] > 2.5 * kn[1:64].mean() and kn[64] > 2.5 * kn[65:448].mean()
    assert abs(k[0, :, 64 + 1:448].mean().item() - 0.5) < 0.02 and abs(k[0, :, 1:64].mean().item()) < 0.02
