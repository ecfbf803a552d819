"""keepkv_decode_attention_static: decode attention for callers that cannot allocate device memory
(code living inside another runtime's memory pool, or a serving loop whose buffers were all fixed at
start-up), so the split-KV scratch is a fixed array inside the library instead of a workspace they
would have had to allocate.  Its results must be those of keepkv_decode_attention.

This file is named so that pytest collects it last: the array is shared, process-wide state, and a
failure here must not hide the results of the other tests in a run that stops at the first failure.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from helpers import HostCache, check_decode_unit, f32_to_dev_bf16, random_cache, to_f64
from paper_2504_09936_b200 import binding as kb


def test_static_scratch_refuses_shapes_beyond_its_size():
    """A shape whose split-KV partials do not fit the built-in array is refused on the host, before
    any CUDA call, with KEEPKV_ERR_WORKSPACE."""
    p = kb.make_params(B=65536, H_q=128, H_kv=16, d=128, N_cap=64)     # 2^20 unit counters + the partial pool > 8 MiB
    dummy = C.c_void_p(256)
    cache = kb.keepkv_cache(256, 256, 256, 256, 256)
    rc = kb.lib().keepkv_decode_attention_static(C.byref(p), C.byref(cache), dummy, dummy, None, 0, dummy, None)
    assert rc == -4 and kb.lib().keepkv_status_string(rc) == b"KEEPKV_ERR_WORKSPACE"


@pytest.mark.gpu
@pytest.mark.parametrize("G,d", [(4, 128), (1, 64)])
def test_static_scratch_decode_matches_workspace_decode_twice(G, d):
    """Two calls in a row (the second finds the first call's leftovers in the shared array) against the
    entry point that uses a caller workspace, on ragged sequences with votes > 1 and a score update."""
    H_kv, B = 2, 5
    p = kb.make_params(B=B, H_q=H_kv * G, H_kv=H_kv, d=d, N_cap=1024, ema_alpha=0.9)
    lens = [1024, 0, 77, 640, 333]
    ref_cache = random_cache(p, lens, seed=31 + G, vote_max=4, scored_frac=0.5)
    new_cache = kb.Cache(ref_cache.K.clone(), ref_cache.V.clone(), ref_cache.votes.clone(), ref_cache.lscore.clone(),
                         ref_cache.seq_len.clone())
    ws, st = kb.new_workspace(p), kb.new_status()
    rng = np.random.default_rng(17)
    for call in range(2):
        q = f32_to_dev_bf16(rng.standard_normal((B, p.H_q, d)).astype(np.float32))
        out_ref, out_new = torch.empty_like(q), torch.empty_like(q)
        lse_ref = torch.empty(B, p.H_q, dtype=torch.float32, device="cuda")
        lse_new = torch.empty_like(lse_ref)
        before = HostCache(new_cache)
        kb.keepkv_decode_attention(p, ref_cache, q, out_ref, lse_ref, True, ws, st)
        kb.keepkv_decode_attention_static(p, new_cache, q, out_new, lse_new, True, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        # the same kernel with the same launch shape, only the scratch lives elsewhere: the same bits
        assert torch.equal(out_new.view(torch.int16), out_ref.view(torch.int16)), f"call {call}: out"
        assert torch.equal(lse_new.view(torch.int32), lse_ref.view(torch.int32)), f"call {call}: lse"
        assert torch.equal(new_cache.lscore.view(torch.int32), ref_cache.lscore.view(torch.int32)), f"call {call}: lscore"
        # ... and the right ones: every unit against the oracle (Eq. 6, Eq. 8), within the decode tolerances
        ls_after = to_f64(new_cache.lscore).reshape(B * H_kv, -1)
        q64, o64, l64 = to_f64(q), to_f64(out_new), to_f64(lse_new)
        for u in range(B * H_kv):
            check_decode_unit(p, u, before, q64, o64, l64, ls_after, what=f"static call {call}")
