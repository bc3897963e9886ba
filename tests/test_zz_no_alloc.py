"""aircache_decode_attn_static, the decode entry point for callers that cannot allocate device memory
(code embedded in another engine's memory pool, or loops that must stay out of the allocator after
start-up): it takes its scratch from an array compiled into the library instead of a caller-provided
workspace.  The test calls it through the C ABI twice in a row, with different queries, and compares each
result with what aircache_decode_attn gives for the same query.  It is collected last on purpose, and it
needs nothing from the other test files, so it also passes when run alone in a fresh process."""
import numpy as np
import pytest
import torch

import paper_2503_23956_b200 as ac
from workloads import Workload, decode_queries, full_cache, window_queries

from harness import GpuPath, logical, rel_row_err

pytestmark = pytest.mark.gpu

TOL = 2e-3
DEV = "cuda:0"


def test_static_scratch_decode_matches_workspace_decode_twice():
    wl = Workload("noalloc", 3, 28, 4, 128, batch=2, n_visual=1000, n_text=40, ratio=0.1, steps=2)
    gp = GpuPath(wl, device=DEV)
    gp.set_full(logical(full_cache(wl, "k", DEV)), logical(full_cache(wl, "v", DEV)))
    gp.score(window_queries(wl, DEV))
    gp.budget()
    gp.compact()
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


def test_static_scratch_rejects_problems_beyond_its_array():
    """A shape whose partial slots would not fit in the built-in array is refused on the host, before anything
    is enqueued (fake pointers: nothing is dereferenced)."""
    sh = ac.shape(1, 1, 128, 8, 128, 64, 8, 4)     # 128 query heads of 128: needs more than 12 MiB
    P = 0x10000000
    rag = ac.Ragged(P, P, P, P, 1000)
    assert ac.aircache_decode_attn_static(sh, rag, P, P, check=False) == ac.ERR_STATIC_SCRATCH
