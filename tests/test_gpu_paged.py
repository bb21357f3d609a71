"""GPU parity of csp_prune_layer_paged: the pass on a cache whose rows live in pages of a pool.  Paging changes
addressing only, so the result must be bit-identical to the dense entry point on the same rows whenever both launches
see the same number of key tiles (the page table pads the logical length to whole pages; a different tile count can
change the cluster size and with it the order in which row statistics are merged: scores then agree to fp32 rounding,
about 2e-7 relative).  It is also compared with the CPU oracle (run on the dense rows) under the tolerances of the pass."""
import numpy as np
import pytest
import torch

import csp_synth as synth
from parity_util import (GpuRun, assert_compaction_exact, assert_index_sets_match, assert_scores_close, bits,
                         gpu_params, orc_params)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def csp():
    from paper_2412_04652_b200 import binding
    binding.lib()
    return binding


def _layouts(lens, seed):
    lays = []
    for i, L in enumerate(lens):
        rng = np.random.RandomState(seed + i)
        img = max(1, min(50, (L - 40) // 2))
        text = L - 2 * img
        cuts = np.sort(rng.randint(0, text - 40 + 1, size=2))
        spans = np.diff(np.concatenate([[0], cuts, [text - 40]])).tolist()
        spans[-1] += 40
        lays.append(synth.interleaved_layout(spans, img))
    return lays


def _paged_copy(k, v, lens, page_rows, seed):
    """Scatters dense [B, H, Lm, d] caches into a shuffled page pool; unused pages hold NaN, unused table
    entries point outside the pool."""
    B, H, Lm, d = k.shape
    per_seq = [-(-int(L) // page_rows) for L in lens]
    max_pages = -(-Lm // page_rows)
    n_pages = sum(per_seq) + 3
    order = np.random.RandomState(seed).permutation(n_pages)
    table = np.full((B, max_pages), 10 ** 6, np.int32)
    k_pool = torch.full((n_pages, H, page_rows, d), float("nan"), dtype=k.dtype, device=k.device)
    v_pool = torch.full((n_pages, H, page_rows, d), float("nan"), dtype=k.dtype, device=k.device)
    nxt = 0
    for b in range(B):
        for i in range(per_seq[b]):
            pg = int(order[nxt]); nxt += 1
            table[b, i] = pg
            r0, r1 = i * page_rows, min((i + 1) * page_rows, int(lens[b]))
            k_pool[pg, :, :r1 - r0] = k[b, :, r0:r1]
            v_pool[pg, :, :r1 - r0] = v[b, :, r0:r1]
    return k_pool, v_pool, torch.from_numpy(table).to(k.device)


@pytest.mark.parametrize("lens,n_q,n_kv,page_rows", [
    ((700, 333, 129), 4, 2, 128),            # ragged batch, one tile per page
    ((1500, 900), 4, 4, 256),                # two tiles per page
    ((1300, 640), 7, 1, 128),                # G = 7: tiles recomputed in the second pass go through the table again
    (tuple(200 + 37 * i for i in range(40)), 8, 8, 128),    # many MHA units: the resident-cluster kernel
    ((5000, 4097), 2, 2, 512),               # long caches, clusters of several CTAs
])
def test_paged_prune_matches_the_dense_one_and_the_oracle(csp, oracle, lens, n_q, n_kv, page_rows):
    cfg = synth.small_config("paged", _layouts(lens, 3), n_q, n_kv, 128, 32, 32, seed=len(lens) + n_q)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    p = gpu_params(csp, cfg)
    mod = cfg.modality()
    dense = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, cfg.budgets).prune()
    assert dense.status() == 0
    k_pool, v_pool, table = _paged_copy(k, v, cfg.seq_lens, page_rows, seed=11)
    pp = gpu_params(csp, cfg)
    pp.max_len = table.shape[1] * page_rows                      # logical length covered by the table
    paged = GpuRun(csp, pp, q, k, v, np.pad(mod, ((0, 0), (0, pp.max_len - mod.shape[1]))), cfg.seq_lens, cfg.budgets)
    csp.prune_layer_paged(pp, paged.q, k_pool, v_pool, table, paged.mod, paged.lens, paged.bud, paged.k_out, paged.v_out,
                          paged.mod_out, paged.n_out, paged.ws, score_self=paged.ss, score_cross=paged.sc, keep_idx=paged.idx)
    assert paged.status() == 0
    assert torch.equal(paged.n_out, dense.n_out) and torch.equal(paged.idx, dense.idx)
    B, H = cfg.batch, cfg.n_kv_heads
    same_tiles = (pp.max_len + 127) // 128 == (cfg.max_len + 127) // 128
    for b in range(B):
        N = int(cfg.seq_lens[b]) - 32
        if same_tiles:
            assert torch.equal(paged.ss[b, :, :N], dense.ss[b, :, :N]) and torch.equal(paged.sc[b, :, :N], dense.sc[b, :, :N])
        else:
            torch.testing.assert_close(paged.ss[b, :, :N], dense.ss[b, :, :N], rtol=2e-6, atol=0)
            torch.testing.assert_close(paged.sc[b, :, :N], dense.sc[b, :, :N], rtol=2e-6, atol=0)
        for h in range(H):
            n = int(dense.n_out[b, h])
            assert torch.equal(paged.k_out[b, h, :n], dense.k_out[b, h, :n])
            assert torch.equal(paged.v_out[b, h, :n], dense.v_out[b, h, :n])
            assert torch.equal(paged.mod_out[b, h, :n], dense.mod_out[b, h, :n])
    # the oracle on the dense rows
    ref = oracle.prune_layer(orc_params(oracle, cfg), q.cpu(), k.cpu(), v.cpu(), mod, cfg.seq_lens, cfg.budgets)
    assert_scores_close(paged.ss.cpu().numpy()[:, :, :cfg.max_len], ref["score_self"], cfg.seq_lens, 32, "self")
    assert_scores_close(paged.sc.cpu().numpy()[:, :, :cfg.max_len], ref["score_cross"], cfg.seq_lens, 32, "cross")
    assert_index_sets_match(paged.idx.cpu().numpy(), paged.n_out.cpu().numpy(), ref, mod, cfg.seq_lens, 32)

    # in place: the kept rows move down inside each sequence's own pages
    kp, vp = k_pool.clone(), v_pool.clone()
    inpl = GpuRun(csp, pp, q, k, v, np.pad(mod, ((0, 0), (0, pp.max_len - mod.shape[1]))), cfg.seq_lens, cfg.budgets)
    csp.prune_layer_paged(pp, inpl.q, kp, vp, table, inpl.mod, inpl.lens, inpl.bud, kp, vp, inpl.mod_out, inpl.n_out, inpl.ws,
                          keep_idx=inpl.idx)
    assert inpl.status() == 0 and torch.equal(inpl.n_out, dense.n_out) and torch.equal(inpl.idx, dense.idx)
    tab = table.cpu().numpy()
    kb, vb = bits(k), bits(v)
    kpb, vpb = bits(kp), bits(vp)
    idx = dense.idx.cpu().numpy()
    for b in range(B):
        for h in range(H):
            n = int(dense.n_out[b, h])
            rows = np.arange(n)
            pg, r = tab[b, rows // page_rows], rows % page_rows
            np.testing.assert_array_equal(kpb[pg, h, r], kb[b, h][idx[b, h, :n]])
            np.testing.assert_array_equal(vpb[pg, h, r], vb[b, h][idx[b, h, :n]])
    assert torch.equal(inpl.mod_out, dense.mod_out)


def test_paged_cache_below_its_budget_is_passed_through(csp, oracle):
    """Algorithm 1's early return on a paged cache: a sequence shorter than its total budget is copied whole, through
    the page table; the other one is pruned.  Supplied log-sum-exp and per-head labels ride along."""
    cfg = synth.small_config("paged", _layouts((600, 300), 9), 4, 2, 128, 32, 32, seed=13)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    total = np.array([100, 301], np.int32)                        # 600 >= 100: pruned; 300 < 301: kept whole
    k_pool, v_pool, table = _paged_copy(k, v, cfg.seq_lens, 128, seed=5)
    p = gpu_params(csp, cfg, cap=300)
    p.max_len = table.shape[1] * 128
    rng = np.random.RandomState(1)
    mod = (rng.rand(2, 2, p.max_len) < 0.4).astype(np.uint8)      # per head
    for b, L in enumerate(cfg.seq_lens):
        mod[b, :, L - 32:L] = 0
    run = GpuRun(csp, p, q, k, v, mod, cfg.seq_lens, cfg.budgets, total_budget=total)
    csp.prune_layer_paged(p, run.q, k_pool, v_pool, table, run.mod, run.lens, run.bud, run.k_out, run.v_out, run.mod_out,
                          run.n_out, run.ws, total_budget=run.tot, score_self=run.ss, score_cross=run.sc, keep_idx=run.idx)
    assert run.status() == 0
    po = orc_params(oracle, cfg, cap=300)
    ref = oracle.prune_layer(po, q.cpu(), k.cpu(), v.cpu(), mod[:, :, :cfg.max_len], cfg.seq_lens, cfg.budgets, total)
    assert (ref["flags"][1] & oracle.FLAG_IDENTITY).all() and not (ref["flags"][0] & oracle.FLAG_IDENTITY).any()
    assert_index_sets_match(run.idx.cpu().numpy(), run.n_out.cpu().numpy(), ref, mod[:, :, :cfg.max_len], cfg.seq_lens, 32)
    assert (run.n_out[1] == 300).all()
    np.testing.assert_array_equal(bits(run.k_out)[1, :, :300], bits(k)[1, :, :300])
    np.testing.assert_array_equal(bits(run.v_out)[1, :, :300], bits(v)[1, :, :300])
    idx = run.idx.cpu().numpy()
    for h in range(2):
        n = int(run.n_out[0, h])
        np.testing.assert_array_equal(bits(run.k_out)[0, h, :n], bits(k)[0, h][idx[0, h, :n]])
        np.testing.assert_array_equal(run.mod_out[0, h, :n].cpu().numpy(), mod[0, h][idx[0, h, :n]])


@pytest.mark.parametrize("G,d,page_rows", [(1, 128, 128), (4, 64, 256), (7, 128, 128)])
def test_decode_over_the_pages_a_prune_in_place_leaves(csp, oracle, G, d, page_rows):
    """Prune a paged cache in place, then one decode query per head attends to what is left, through the same page
    table: compared with the dense decode call on the dense prune's output (bit-identical: the same rows in the same
    order) and with the oracle."""
    lens = (900, 517, 1300)
    cfg = synth.small_config("paged", _layouts(lens, 21), 2 * G, 2, d, 32, 32, seed=30 + G)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    p = gpu_params(csp, cfg)
    dense = GpuRun(csp, p, q, k, v, cfg.modality(), cfg.seq_lens, cfg.budgets).prune()
    k_pool, v_pool, table = _paged_copy(k, v, cfg.seq_lens, page_rows, seed=3)
    pp = gpu_params(csp, cfg)
    pp.max_len = table.shape[1] * page_rows
    inpl = GpuRun(csp, pp, q, k, v, np.pad(cfg.modality(), ((0, 0), (0, pp.max_len - cfg.max_len))), cfg.seq_lens, cfg.budgets)
    csp.prune_layer_paged(pp, inpl.q, k_pool, v_pool, table, inpl.mod, inpl.lens, inpl.bud, k_pool, v_pool, inpl.mod_out,
                          inpl.n_out, inpl.ws)
    assert inpl.status() == 0 and torch.equal(inpl.n_out, dense.n_out)
    gen = torch.Generator(device="cuda").manual_seed(5)
    q1 = torch.randn(3, 2 * G, d, device="cuda", generator=gen).to(torch.bfloat16)
    cap = p.out_capacity
    pd = csp.Params(3, 2 * G, 2, d, 1, 0, cap, cap)
    out_dense, out_paged = torch.zeros(3, 2 * G, d, device="cuda"), torch.full((3, 2 * G, d), 9.0, device="cuda")
    wd = csp.new_decode_workspace(pd)
    csp.decode_attn(pd, q1, dense.k_out, dense.v_out, dense.n_out, out_dense, wd)
    csp.decode_attn_paged(pd, q1, k_pool, v_pool, table, inpl.n_out, out_paged, wd)
    assert csp.device_status(wd) == 0
    assert torch.equal(out_paged, out_dense)
    po = oracle.Params(3, 2 * G, 2, d, 1, 0, cap, cap, dtype=oracle.BF16)
    want = oracle.decode_attn(po, q1.cpu(), dense.k_out.cpu(), dense.v_out.cpu(), dense.n_out.cpu().numpy())
    got = out_paged.cpu().numpy().astype(np.float64)
    tol = 2e-3 * np.abs(want) + 1e-5 * float(v.float().abs().max())
    assert (np.abs(got - want) <= tol).all()
    bad = table.clone()
    bad[1, 0] = -5
    csp.decode_attn_paged(pd, q1, k_pool, v_pool, bad, inpl.n_out, out_paged, wd)
    assert csp.device_status(wd) & csp.DEV_BAD_LEN


def test_paged_arguments_are_checked_and_a_bad_page_is_flagged(csp):
    cfg = synth.small_config("paged", _layouts((300, 200), 5), 2, 2, 128, 32, 32, seed=9)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    k_pool, v_pool, table = _paged_copy(k, v, cfg.seq_lens, 128, seed=1)
    p = gpu_params(csp, cfg)
    p.max_len = table.shape[1] * 128
    run = GpuRun(csp, p, q, k, v, np.pad(cfg.modality(), ((0, 0), (0, p.max_len - cfg.max_len))), cfg.seq_lens, cfg.budgets)

    def call(pool_k, tab, params=p):
        csp.prune_layer_paged(params, run.q, pool_k, v_pool, tab, run.mod, run.lens, run.bud, run.k_out, run.v_out,
                              run.mod_out, run.n_out, run.ws)
    with pytest.raises(csp.CspError) as e:                       # pages must hold whole 128-key tiles
        call(k_pool[:, :, :64], table)
    assert e.value.code == csp.ERR_INVALID_ARG
    with pytest.raises(csp.CspError) as e:                       # the table must cover max_len
        call(k_pool, table[:, :1].contiguous())
    assert e.value.code == csp.ERR_INVALID_ARG
    bad = table.clone()
    bad[0, 1] = 10 ** 6                                          # a page number outside the pool, inside the sequence
    call(k_pool, bad)
    assert run.status() & csp.DEV_BAD_LEN
    call(k_pool, table)                                          # and the context is still usable
    assert run.status() == 0
