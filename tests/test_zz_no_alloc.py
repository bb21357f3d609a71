"""The allocation-free entry point, csp_prune_layer_static, against csp_prune_layer.

Some users of this library cannot give it a workspace: their process has already handed all device
memory to another allocator, or they sit in a place where allocating is not allowed.  For them the
library carries its own fixed scratch array.  This test calls that entry point through the C
interface twice in a row (the array is shared between calls and keeps old contents, so the second
call must not be disturbed by the first) and requires the same result as the ordinary entry point
with a caller-allocated workspace: identical row counts and bit-identical compacted K, V and labels,
which is the bar the other GPU tests use for this data.  The second call is also checked for what the
entry point is for: neither the driver's free-memory figure nor torch's allocator moves across it.  The
kept rows are compared with the CPU oracle as well.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import csp_synth as synth

pytestmark = pytest.mark.gpu


def _inputs(csp, seed, lens):
    lays = [synth.interleaved_layout([30, 45, L - 2 * 60 - 75], 60) for L in lens]
    cfg = synth.small_config("static", lays, 4, 2, 128, 32, 32, seed=seed, visual_pct=40, text_pct=30)
    q, k, v = synth.make_layer(cfg, 0, "cuda")
    cap = cfg.out_capacity()
    p = csp.Params(cfg.batch, 4, 2, 128, 32, 32, cfg.max_len, cap)
    dev = dict(mod=torch.from_numpy(cfg.modality()).cuda(), lens=torch.from_numpy(cfg.seq_lens).cuda(),
               bud=torch.from_numpy(cfg.budgets).cuda())
    return cfg, p, q, k, v, dev


def _outputs(p, dtype):
    B, H, cap, d = p.batch, p.n_kv_heads, p.out_capacity, p.head_dim
    return dict(k_out=torch.zeros(B, H, cap, d, dtype=dtype, device="cuda"),
                v_out=torch.zeros(B, H, cap, d, dtype=dtype, device="cuda"),
                mod_out=torch.zeros(B, H, cap, dtype=torch.uint8, device="cuda"),
                n_out=torch.full((B, H), -7, dtype=torch.int32, device="cuda"))


def test_static_entry_point_matches_workspace_entry_point_twice(oracle):
    assert torch.cuda.is_available()
    from paper_2412_04652_b200 import binding as csp
    assert csp.static_workspace_limit() == 8 << 20
    for call, (seed, lens) in enumerate([(3, (700, 410)), (4, (333, 900))]):     # two calls in a row, new data
        cfg, p, q, k, v, dev = _inputs(csp, seed, lens)
        want, got = _outputs(p, k.dtype), _outputs(p, k.dtype)
        ws = csp.new_workspace(p)
        csp.prune_layer(p, q, k, v, dev["mod"], dev["lens"], dev["bud"], want["k_out"], want["v_out"],
                        want["mod_out"], want["n_out"], ws)
        assert csp.device_status(ws) == 0
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        csp.prune_layer_static(p, q, k, v, dev["mod"], dev["lens"], dev["bud"], got["k_out"], got["v_out"],
                               got["mod_out"], got["n_out"], dev_status_out=status)
        torch.cuda.synchronize()
        if call == 1:       # the first call on a device may load the kernels' code; the second finds all in place
            assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == held_before
        assert int(status.item()) == 0, f"call {call}: device status {int(status.item())}"
        assert torch.equal(got["n_out"], want["n_out"]) and int(want["n_out"].min()) > 32
        for b in range(p.batch):
            for h in range(p.n_kv_heads):
                n = int(want["n_out"][b, h])
                for name in ("k_out", "v_out", "mod_out"):
                    assert torch.equal(got[name][b, h, :n], want[name][b, h, :n]), (call, name, b, h)
        # and against the CPU oracle: same row counts; where the kept sets agree, the same bytes
        op = oracle.Params(p.batch, 4, 2, 128, 32, 32, cfg.max_len, p.out_capacity)
        ref = oracle.prune_layer(op, q.cpu(), k.cpu(), v.cpu(), cfg.modality(), cfg.seq_lens, cfg.budgets)
        np.testing.assert_array_equal(got["n_out"].cpu().numpy(), ref["n_out"])
        ko = got["k_out"].cpu().view(torch.int16).numpy().view(np.uint16)
        mo = got["mod_out"].cpu().numpy()
        same_rows = 0
        for b in range(p.batch):
            for h in range(p.n_kv_heads):
                n = int(ref["n_out"][b, h])
                np.testing.assert_array_equal(mo[b, h, n - 32:n], ref["mod_out"][b, h, n - 32:n])
                np.testing.assert_array_equal(ko[b, h, n - 32:n], ref["k_out"][b, h, n - 32:n])     # the recent block
                theirs = {r.tobytes() for r in ref["k_out"][b, h, :n]}
                same_rows += sum(r.tobytes() in theirs for r in ko[b, h, :n])
        total_rows = int(ref["n_out"].sum())
        assert same_rows >= total_rows - 8, "kept rows differ from the oracle's beyond a few boundary ties"


def test_static_entry_point_refuses_shapes_beyond_its_scratch():
    from paper_2412_04652_b200 import binding as csp
    p = csp.Params(8, 32, 32, 128, 32, 32, 8192, 2048)     # workspace far above 8 MiB
    assert csp.workspace_bytes(p) > csp.static_workspace_limit()
    z = torch.zeros(1, 1, 1, 128, dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(1, 1, dtype=torch.uint8, device="cuda")
    i = torch.zeros(8, 4, dtype=torch.int32, device="cuda")
    with pytest.raises(csp.CspError) as err:
        csp.prune_layer_static(p, z, z, z, m, i, i, z, z, None, i)
    assert err.value.code == csp.ERR_WORKSPACE
