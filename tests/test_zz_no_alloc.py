"""The allocation-free greedy-token call against the tokens vlac_step itself picks.

Some users of this library may not allocate device memory while their loop runs (memory reserved
once at start-up, or a GPU whose memory is owned by a single pool).  For them the library offers
``vlac_greedy_tokens_static``, whose only scratch is an array inside the library image.  This test
calls it through the C ABI on the logits two consecutive control steps produced and requires the
very tokens those steps reported (integers: no tolerance), so it also covers the second call
finding the first call's leftovers in the shared array.  It lives in a file collected last so that
a run stopping at the first failure has already exercised everything else.
"""
import numpy as np
import pytest
import torch

from paper_2502_02175_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_greedy_tokens_match_step_tokens_twice():
    from paper_2502_02175_b200 import binding as vb
    cfg = synth.tiny_config()
    model = synth.make_model(cfg, 4)
    dev = vb.DeviceModel(model)
    ctx = vb.vlac_create(vb.make_config(cfg, 2), dev.weights)
    cache = vb.vlac_cache_alloc(ctx, 2)
    try:
        ids = torch.from_numpy(synth.make_prompt_ids(cfg, 4, batch=2)).to("cuda")
        rng = np.random.default_rng(4)
        feats = vb.upload_bf16(synth.f32_to_bf16(rng.standard_normal((2, cfg.n_vision, cfg.hidden), dtype=np.float32)))
        pairs = [synth.rerandomised_pair(cfg, 40 + b, 13) for b in range(2)]
        params, keep = vb.make_params(top_k=32, alpha_override=[0.5, 1.0])
        for step in range(2):                                     # cold step, then a cached step
            frames = torch.from_numpy(np.stack([p[step] for p in pairs])).to("cuda")
            want = torch.zeros((2, cfg.n_action), dtype=torch.int32, device="cuda")
            logits = torch.zeros((2, cfg.n_action, cfg.vocab), dtype=torch.float32, device="cuda")
            vb.vlac_step(ctx, cache, frames, feats, ids, params, False, want, logits)
            got = torch.full((2 * cfg.n_action,), -1, dtype=torch.int32, device="cuda")
            vb.vlac_greedy_tokens_static(logits.view(2 * cfg.n_action, cfg.vocab), got)
            torch.cuda.synchronize()
            assert torch.equal(got.view(2, cfg.n_action), want), (step, got, want)
        # ties go to the lower index; strided rows are honoured
        x = torch.zeros((3, 100), dtype=torch.float32, device="cuda")
        x[0, 7] = x[0, 50] = 2.0
        x[1, 99] = 1.0
        x[2] = -1.0
        got = torch.zeros(3, dtype=torch.int32, device="cuda")
        vb.vlac_greedy_tokens_static(x[:, :60], got)
        torch.cuda.synchronize()
        assert got.tolist() == [7, 0, 0]
        # -0.0 and +0.0 are equal: the lower index wins
        z = torch.full((1, 16), -1.0, dtype=torch.float32, device="cuda")
        z[0, 3] = -0.0
        z[0, 9] = 0.0
        got1 = torch.zeros(1, dtype=torch.int32, device="cuda")
        vb.vlac_greedy_tokens_static(z, got1)
        torch.cuda.synchronize()
        assert got1.tolist() == [3]
        # nothing is allocated: the free device memory is the same before and after a (warmed-up) call
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        vb.vlac_greedy_tokens_static(x[:, :60], got)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
        # bad arguments are refused before anything is launched
        import ctypes as C
        assert vb.lib.vlac_greedy_tokens_static(None, 1, 8, 8, got.data_ptr(), None) == -1
        assert vb.lib.vlac_greedy_tokens_static(x.data_ptr(), 1, 8, 8, None, None) == -1
        assert vb.lib.vlac_greedy_tokens_static(x.data_ptr(), 1, 100, 60, got.data_ptr(), None) == -1      # row_stride < vocab
        assert vb.lib.vlac_greedy_tokens_static(x.data_ptr(), 0, 8, 8, got.data_ptr(), None) == -1
        # capacity is enforced with its own error code and nothing runs
        big = torch.zeros((65, 8), dtype=torch.float32, device="cuda")
        out = torch.zeros(65, dtype=torch.int32, device="cuda")
        with pytest.raises(vb.VlacError) as e:
            vb.vlac_greedy_tokens_static(big, out)
        assert e.value.status == -6
    finally:
        vb.vlac_cache_free(cache)
        vb.vlac_destroy(ctx)
