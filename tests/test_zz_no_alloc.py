"""aircache_decode_attn_static, the decode entry point for callers that cannot allocate device memory
(code embedded in another engine's memory pool, or loops that must stay out of the allocator after
start-up): it takes its scratch from an array compiled into the library instead of a caller-provided
workspace.  The test calls it through the C ABI twice in a row, with different queries, and compares each
result with what aircache_decode_attn gives for the same query and with the CPU oracle's attention over the
same compressed cache.  It is collected last on purpose, and it needs nothing from the other test files, so
it also passes when run alone in a fresh process."""
import numpy as np
import pytest
import torch

import paper_2503_23956_b200 as ac
from workloads import Workload, decode_queries, full_cache, window_queries

from harness import GpuPath, logical, oracle_dims, rel_row_err, u16

pytestmark = pytest.mark.gpu

TOL = 2e-3
DEV = "cuda:0"


def test_static_scratch_decode_matches_workspace_decode_twice(oracle_mod):
    wl = Workload("noalloc", 3, 28, 4, 128, batch=2, n_visual=1000, n_text=40, ratio=0.1, steps=2)
    gp = GpuPath(wl, device=DEV)
    gp.set_full(logical(full_cache(wl, "k", DEV)), logical(full_cache(wl, "v", DEV)))
    gp.score(window_queries(wl, DEV))
    gp.budget()
    gp.compact()
    dm = oracle_dims(oracle_mod, wl)
    kc, vc = u16(gp.k_c), u16(gp.v_c)
    offs, lens = gp.offsets.cpu().numpy(), gp.lens.cpu().numpy()
    out_static = torch.empty_like(gp.out)
    for step in range(2):
        q = decode_queries(wl, step, DEV)
        gp.out.fill_(float("nan"))
        gp.decode(q)
        assert gp.status() == 0
        want = gp.out.cpu().numpy()
        assert np.isfinite(want).all()
        out_static.fill_(float("nan"))
        ac.aircache_decode_attn_static(gp.sh, gp.cache, q, out_static)
        torch.cuda.synchronize()
        got = out_static.cpu().numpy()
        assert np.isfinite(got).all()
        assert rel_row_err(got, want) <= TOL
        assert rel_row_err(got, oracle_mod.decode(dm, kc, vc, offs, lens, u16(q), wl.scale)) <= TOL


def test_static_scratch_rejects_problems_beyond_its_array():
    """A shape whose partial slots would not fit in the built-in array is refused on the host, before anything
    is enqueued (fake pointers: nothing is dereferenced)."""
    sh = ac.shape(1, 1, 128, 8, 128, 64, 8, 4)     # 128 query heads of 128: needs more than 12 MiB
    P = 0x10000000
    rag = ac.Ragged(P, P, P, P, 1000)
    assert ac.aircache_decode_attn_static(sh, rag, P, P, check=False) == ac.ERR_STATIC_SCRATCH


def _static_need(sms, n_q_heads, head_dim):
    """Bytes of the built-in array a problem takes (the rule stated in include/aircache.h)."""
    slot_floats = (n_q_heads * (head_dim + 2) + 3) // 4 * 4
    return 256 + 1792 * 4 + 2 * min(sms, 256) * slot_floats * 4


def test_static_scratch_limit_is_where_the_header_says(oracle_mod):
    """The largest head count (8 KV heads, head_dim 128) whose scratch fits the array decodes correctly, the next
    one up is refused - both computed from this GPU's SM count with the header's formula."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    limit = 12 * 1024 * 1024
    fits = [hq for hq in range(8, 129, 8) if _static_need(sms, hq, 128) <= limit]
    assert fits and fits[-1] < 128
    hq_ok, hq_over = fits[-1], fits[-1] + 8
    P = 0x10000000
    rag = ac.Ragged(P, P, P, P, 1000)
    assert ac.aircache_decode_attn_static(ac.shape(1, 1, hq_over, 8, 128, 64, 8, 4), rag, P, P,
                                          check=False) == ac.ERR_STATIC_SCRATCH
    wl = Workload("noalloc_wide", 2, hq_ok, 8, 128, batch=1, n_visual=3000, n_text=24, ratio=0.5, steps=1, window=4)
    gp = GpuPath(wl, device=DEV)
    gp.set_full(logical(full_cache(wl, "k", DEV)), logical(full_cache(wl, "v", DEV)))
    gp.score(window_queries(wl, DEV))
    gp.budget()
    gp.compact()
    q = decode_queries(wl, 0, DEV)
    out = torch.full_like(gp.out, float("nan"))
    ac.aircache_decode_attn_static(gp.sh, gp.cache, q, out)
    torch.cuda.synchronize()
    want = oracle_mod.decode(oracle_dims(oracle_mod, wl), u16(gp.k_c), u16(gp.v_c), gp.offsets.cpu().numpy(),
                             gp.lens.cpu().numpy(), u16(q), wl.scale)
    assert rel_row_err(out.cpu().numpy(), want) <= TOL
