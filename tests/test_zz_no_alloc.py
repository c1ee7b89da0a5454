"""The allocation-free FFN entry point (saem_expert_ffn_static) against saem_expert_ffn.

Some callers of this library cannot allocate device memory (the memory pool belongs to a host
application, or an allocation inside their loop is not allowed), so they have no workspace to
give.  This entry point keeps its only scratch -- the hidden activations -- in a fixed array
inside the library.  The test calls it twice in a row through the C ABI on different inputs (the
array keeps the first call's contents) and compares each result with the regular entry point's
and with the CPU oracle's.
It is collected last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2608_21614_b200 import inputs as gen

pytestmark = pytest.mark.gpu


def test_static_scratch_ffn_matches_regular_entry_point_twice(oracle):
    import gpu_util as g
    from paper_2608_21614_b200 import binding as B
    from paper_2608_21614_b200.layer import MoELayer

    cfg = gen.layer_config("c1")                       # d 512, f 1024, 8 experts, top-2, 64 tokens
    li = gen.layer_inputs(cfg)
    T, k, d, f, E = cfg.tokens, cfg.top_k, cfg.d_model, cfg.d_ff, cfg.n_experts
    layer = MoELayer(d, f, E, k, T)
    layer.load_all(li.gate, li.up, li.down)
    layer.copy_stream.synchronize()
    rng = np.random.default_rng(123)
    for call in range(2):
        logits = li.logits if call == 0 else rng.standard_normal((T, E)).astype(np.float32)
        x = li.x if call == 0 else gen.activations(rng, T, d)
        layer.route(g.dev(logits), T)
        layer.repack(g.dev(x), T)
        layer.expert_ffn(T)                             # the existing entry point
        y_static = torch.full((T * k, d), float("nan"), dtype=torch.float32, device="cuda:0")
        B.saem_expert_ffn_static(layer.x_packed, layer.offsets, E, T * k, d, f, layer.ctx.slot_ptr, y_static)
        torch.cuda.synchronize()
        g.assert_close(g.host(y_static), g.host(layer.y_packed), "static vs regular, call %d" % call)
        # ... and against the CPU oracle directly, so that a mistake shared by both GPU paths cannot hide
        off = g.host(layer.offsets)[:E + 1]
        y_ref = oracle.expert_ffn(g.host(layer.x_packed[:T * k]), off, li.gate, li.up, li.down)
        g.assert_close(g.host(y_static), y_ref, "static vs oracle, call %d" % call)
    # max_rows below the last offset: the rows from max_rows on are left untouched
    cut = int(off[E - 1]) + 1 if off[E] - off[E - 1] > 1 else T * k - 3
    y_cut = torch.full((T * k, d), float("nan"), dtype=torch.float32, device="cuda:0")
    B.saem_expert_ffn_static(layer.x_packed, layer.offsets, E, cut, d, f, layer.ctx.slot_ptr, y_cut)
    torch.cuda.synchronize()
    g.assert_close(g.host(y_cut[:cut]), y_ref[:cut], "static, max_rows inside the last segment")
    assert torch.isnan(y_cut[cut:]).all()
    # sizes beyond the fixed array are refused before anything is enqueued
    too_many = B.SAEM_STATIC_SCRATCH_ELEMS // f + 1
    code = B.saem_expert_ffn_static(layer.x_packed, layer.offsets, E, too_many, d, f, layer.ctx.slot_ptr,
                                    layer.y_packed, check=False)
    assert code == B.SAEM_ERR_WORKSPACE
    assert layer.device_status() == 0
    layer.close()
