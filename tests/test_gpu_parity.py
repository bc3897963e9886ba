"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element, on the same seeded
inputs.  Integer results (elite masks, budgets, offsets, kept-token lists, gathered bytes) must be equal;
floating-point results must agree within 2e-3 (scores: element-wise relative; attention outputs: per row,
max |a - b| / max |b|).  Stage-isolated tests feed a CUDA stage the oracle's upstream output, so the
integer stages are compared on identical input bits; end-to-end tests chain the CUDA stages."""
import numpy as np
import pytest
import torch

from workloads import CONFIGS, Workload, decode_queries

from harness import GpuPath, gen_inputs, logical, oracle_dims, rel_elem_err, rel_row_err, shape_of, u16

pytestmark = pytest.mark.gpu

TOL = 2e-3
DEV = "cuda:0"


def small(name, L=3, Hq=28, Hkv=4, d=128, B=2, Nv=1000, Nt=40, ratio=0.1, W=16, **kw):
    return Workload(name, L, Hq, Hkv, d, batch=B, n_visual=Nv, n_text=Nt, ratio=ratio, steps=2, window=W, **kw)


CASES = {
    "c1": CONFIGS["c1"],
    "s7b": small("s7b"),                                           # 7B head layout, ragged tails everywhere
    "s72b": small("s72b", L=2, Hq=64, Hkv=8, B=2, Nv=777, Nt=33),   # 72B head layout
    "mha64": small("mha64", L=2, Hq=4, Hkv=4, d=64, B=3, Nv=300, Nt=20, W=8),
    "g16": small("g16", L=2, Hq=16, Hkv=1, d=64, B=2, Nv=257, Nt=17, W=5),   # 16 query heads per KV head
    "kv2": small("kv2", L=2, Hq=12, Hkv=2, d=128, B=2, Nv=515, Nt=64, W=64),  # widest window
    "kv1": small("kv1", L=2, Hq=3, Hkv=1, d=128, B=1, Nv=130, Nt=9, W=9),
    # the paper's own window: every text token a candidate (W = N_t = 128: two mask words per head)
    "w128": small("w128", L=2, Hq=28, Hkv=4, d=128, B=1, Nv=700, Nt=128, W=128),
    "w100": small("w100", L=1, Hq=8, Hkv=2, d=64, B=2, Nv=300, Nt=100, W=100),
    # the window's text keys take a share of the softmax that differs by layer: the strength term of Eq. 11 moves
    # the budgets (on the other cases the visual tokens hold nearly all of the mass in every layer)
    "textmass": small("textmass", L=6, B=1, Nv=600, Nt=32, text_amp_hi=8.0),
    # long regions cut across many CTAs with an odd head count (padded partial slots, multi-round merge)
    "kv1long": small("kv1long", L=2, Hq=3, Hkv=1, d=128, B=1, Nv=9000, Nt=9, W=4, ratio=0.9),
    # more (region, KV head) pairs than SMs: the by-region decode schedule with several regions per CTA
    "many": small("many", L=10, Hq=28, Hkv=4, d=128, B=4, Nv=300, Nt=20, W=8),
    # the largest number of regions the library takes (L * B = 1792), each of them tiny
    "maxreg": small("maxreg", L=28, Hq=8, Hkv=2, d=64, B=64, Nv=40, Nt=4, W=4, ratio=0.25),
}


@pytest.fixture(scope="module")
def oracle(oracle_mod):
    return oracle_mod


def cpu_inputs(wl):
    return gen_inputs(wl, "cpu")


_ORACLE_CACHE = {}


def oracle_path(oracle, wl, ratio=None, alpha=None, slack=0, mode=0):
    """Chained oracle: scores -> moments -> budgets -> compact.  Cached per argument tuple."""
    key = (wl, ratio, alpha, slack, mode)
    if key in _ORACLE_CACHE:
        return _ORACLE_CACHE[key]
    ratio = wl.ratio if ratio is None else ratio
    alpha = wl.alpha if alpha is None else alpha
    k, v, qw = cpu_inputs(wl)
    dm = oracle_dims(oracle, wl)
    kl, vl = u16(logical(k)), u16(logical(v))
    sc = oracle.score(dm, kl, u16(qw), wl.scale, alpha)
    st, sk = oracle.moments(sc["scores"])
    bud = oracle.allocate(st, sk, wl.n_visual, ratio, mode)
    cp = oracle.compact(dm, slack, kl, vl, sc["scores"], bud)
    res = dict(k=k, v=v, qw=qw, dims=dm, scores=sc["scores"], mask=sc["elite_mask"], strength=st, skew=sk,
               budgets=bud, compact=cp, ratio=ratio, alpha=alpha)
    _ORACLE_CACHE[key] = res
    return res


def make_gpu(wl, ref, slack=0):
    gp = GpuPath(wl, ratio=ref["ratio"], device=DEV, slack=slack)
    gp.set_full(logical(ref["k"].to(DEV)), logical(ref["v"].to(DEV)))
    return gp


def compare_cache(gp, cp):
    """Valid rows of K'/V', offsets, lens and kept lists are bit-identical to the oracle's."""
    assert np.array_equal(gp.offsets.cpu().numpy(), cp["offsets"])
    assert np.array_equal(gp.lens.cpu().numpy(), cp["lens"])
    kc, vc = u16(gp.k_c), u16(gp.v_c)
    for r in range(len(cp["lens"])):
        a, n = int(cp["offsets"][r]), int(cp["lens"][r])
        assert np.array_equal(kc[a:a + n], cp["k"][a:a + n]), f"K' region {r}"
        assert np.array_equal(vc[a:a + n], cp["v"][a:a + n]), f"V' region {r}"


# --------------------------------------------------------------------------------------------------
# stage-isolated parity
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("alpha", [0.9, 0.0, 1.0])
def test_score_parity(oracle, case, alpha):
    wl = CASES[case]
    ref = oracle_path(oracle, wl, alpha=alpha)
    gp = make_gpu(wl, ref)
    gp.score(ref["qw"].to(DEV), alpha=alpha)
    assert gp.status() == 0
    mask = gp.mask.cpu().numpy().view(np.uint64)
    assert np.array_equal(mask, ref["mask"]), "elite sets differ"
    err = rel_elem_err(gp.scores.cpu().numpy(), ref["scores"])
    assert err <= TOL, err


def test_score_parity_sequence_longer_than_the_one_pass_kernel_takes(oracle):
    """The one-pass scoring kernel lets the blocks of a KV group wait for one another, so the library only uses
    it while a group's blocks (one per 512 visual keys) are at most half of the blocks the GPU holds at once;
    200 000 visual tokens are beyond that on any GPU of today (391 blocks per group against at most 370), and
    the call takes the two-kernel form (statistics pass, then importance pass) instead."""
    wl = small("verylong", L=1, Hq=2, Hkv=1, d=64, B=1, Nv=200_000, Nt=16, W=8)
    ref = oracle_path(oracle, wl, alpha=0.9)
    gp = make_gpu(wl, ref)
    gp.score(ref["qw"].to(DEV), alpha=0.9)
    assert gp.status() == 0
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"]), "elite sets differ"
    err = rel_elem_err(gp.scores.cpu().numpy(), ref["scores"])
    assert err <= TOL, err


@pytest.mark.parametrize("seed", range(12))
def test_score_parity_random_mid_size_shapes(oracle, seed):
    """Seeded random shapes with thousands of visual tokens (several key chunks per KV group, ragged tails), head
    layouts from 1 to 8 KV heads and 1 to 16 heads per group, windows up to the whole text, thresholds that give
    from one to over a hundred elite rows per group, per layer and per KV head: masks equal, scores within the
    tolerance."""
    rng = np.random.default_rng(1000 + seed)
    hkv, g, d = int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2, 4, 7, 8, 16])), int(rng.choice([64, 128]))
    L, B = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    nv, nt = int(rng.integers(300, 9000)), int(rng.integers(16, 130))
    W = int(rng.integers(1, min(nt, 128) + 1))
    alpha = float(rng.choice([0.9, 0.9, 0.5, 0.1, 1e-3, 0.99]))
    per_kv_head = seed % 2
    wl = small(f"mid{seed}", L=L, Hq=hkv * g, Hkv=hkv, d=d, B=B, Nv=nv, Nt=nt, W=W, alpha=alpha)
    k, v, qw = cpu_inputs(wl)
    dm = oracle_dims(oracle, wl)
    fn = oracle.score_groups if per_kv_head else oracle.score
    sc = fn(dm, u16(logical(k)), u16(qw), wl.scale, alpha)
    gp = GpuPath(wl, device=DEV, per_kv_head=per_kv_head)
    gp.set_full(logical(k.to(DEV)), logical(v.to(DEV)))
    gp.score(qw.to(DEV), alpha=alpha)
    assert gp.status() == 0
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64).reshape(-1), sc["elite_mask"].reshape(-1)), wl
    err = rel_elem_err(gp.scores.cpu().numpy().reshape(-1), sc["scores"].reshape(-1))
    assert err <= TOL, (wl, err)


@pytest.mark.parametrize("case", ["kv2", "s7b", "g16", "w128"])
def test_score_parity_many_elite_rows_below_the_dense_threshold(oracle, case):
    """A small but non-zero threshold makes almost every candidate elite (hundreds of rows per KV group on the
    widest window) while the launch stays on the sparse-window kernels: their loops over slabs of rows run more
    than once, and the wide instantiation of the statistics pass does the work."""
    wl = CASES[case]
    alpha = 1e-4
    ref = oracle_path(oracle, wl, alpha=alpha)
    rows = [bin(int(m)).count("1") for m in ref["mask"].ravel()]
    assert max(rows) * wl.group > 64 or case != "kv2"      # the case is what it claims to be
    gp = make_gpu(wl, ref)
    gp.score(ref["qw"].to(DEV), alpha=alpha)
    assert gp.status() == 0
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"]), "elite sets differ"
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL


@pytest.mark.parametrize("alpha", [0.9, 0.0])
@pytest.mark.parametrize("layout", ["head_major", "layer_innermost"])
def test_score_parity_other_cache_layouts(oracle, alpha, layout):
    """The same scores from a head-major cache [L,B,Hkv,N,d] and from one whose layer stride is the smallest
    ([B,Hkv,N,L,d] storage): the kernels (and, for alpha = 0, the tensor map of the dense path) only see strides."""
    wl = CASES["s7b"]
    ref = oracle_path(oracle, wl, alpha=alpha)
    kl, vl = logical(ref["k"]), logical(ref["v"])                      # logical [L,B,Hkv,N,d]
    if layout == "head_major":
        kd, vd = kl.contiguous().to(DEV), vl.contiguous().to(DEV)
    else:
        kd = kl.permute(1, 2, 3, 0, 4).contiguous().to(DEV).permute(3, 0, 1, 2, 4)
        vd = vl.permute(1, 2, 3, 0, 4).contiguous().to(DEV).permute(3, 0, 1, 2, 4)
    gp = GpuPath(wl, ratio=ref["ratio"], device=DEV)
    gp.set_full(kd, vd)
    gp.score(ref["qw"].to(DEV), alpha=alpha)
    assert gp.status() == 0
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"])
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL
    gp.budget()
    gp.compact()
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
    compare_cache(gp, ref["compact"])


@pytest.mark.parametrize("case", ["c1", "s7b", "mha64"])
@pytest.mark.parametrize("mode", [0, 1, 2, 3])
@pytest.mark.parametrize("ratio", [0.1, 0.83])
def test_budget_parity_on_oracle_scores(oracle, case, mode, ratio):
    wl = CASES[case]
    ref = oracle_path(oracle, wl, ratio=ratio, mode=mode, slack=3)
    gp = make_gpu(wl, ref, slack=3)
    gp.budget(scores=torch.from_numpy(ref["scores"]).to(DEV), mode=mode)
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
    assert np.allclose(gp.strength.cpu().numpy(), ref["strength"], rtol=1e-12, atol=0)
    assert np.allclose(gp.skew.cpu().numpy(), ref["skew"], rtol=1e-9, atol=1e-12)
    assert np.array_equal(gp.offsets.cpu().numpy(), ref["compact"]["offsets"])
    assert np.array_equal(gp.lens.cpu().numpy(), ref["compact"]["lens"])
    assert int(gp.budgets.sum()) == wl.batch * oracle.total_kept(wl.n_visual, wl.n_layers, ratio)


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("slack", [0, 5])
def test_compact_parity_on_oracle_scores_and_budgets(oracle, case, slack):
    wl = CASES[case]
    ref = oracle_path(oracle, wl, slack=slack)
    gp = make_gpu(wl, ref, slack=slack)
    gp.budget(scores=torch.from_numpy(ref["scores"]).to(DEV))   # layout (offsets, lens) comes from the budget call
    gp.compact(scores=torch.from_numpy(ref["scores"]).to(DEV), budgets=torch.from_numpy(ref["budgets"]).to(DEV))
    assert np.array_equal(gp.kept.cpu().numpy()[:len(ref["compact"]["kept_idx"])], ref["compact"]["kept_idx"])
    compare_cache(gp, ref["compact"])


@pytest.mark.parametrize("n_visual", [8195, 41000])
def test_select_long_regions(oracle, n_visual):
    """The shared-memory and the re-reading variants of the select (more than 8192 / 40960 visual tokens),
    on duplicated scores."""
    wl = small("sel_long", L=2, Hq=2, Hkv=1, d=64, B=1, Nv=n_visual, Nt=4, W=2, ratio=0.3)
    rng = np.random.default_rng(n_visual)
    k, v, _ = cpu_inputs(wl)
    scores = (rng.integers(0, 1000, size=(wl.n_layers, wl.batch, wl.n_visual)) / 1024.0).astype(np.float32)
    dm = oracle_dims(oracle, wl)
    T = oracle.total_kept(wl.n_visual, wl.n_layers, wl.ratio)
    budgets = np.array([[T // 3], [T - T // 3]], np.int32)
    cp = oracle.compact(dm, 0, u16(logical(k)), u16(logical(v)), scores, budgets)
    gp = GpuPath(wl, device=DEV)
    gp.set_full(logical(k.to(DEV)), logical(v.to(DEV)))
    gp.offsets.copy_(torch.from_numpy(cp["offsets"])); gp.lens.copy_(torch.from_numpy(cp["lens"]))
    gp.compact(scores=torch.from_numpy(scores).to(DEV), budgets=torch.from_numpy(budgets).to(DEV))
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)


def test_select_ties_zero_and_full_budgets(oracle):
    """Heavily duplicated scores (ties broken by the lower index), a layer that keeps nothing and one that
    keeps everything, negative zero and denormal scores; head-major source layout."""
    wl = small("ties", L=4, Hq=8, Hkv=2, d=64, B=2, Nv=611, Nt=12, W=4)
    rng = np.random.default_rng(7)
    k, v, _ = cpu_inputs(wl)
    scores = (rng.integers(0, 6, size=(wl.n_layers, wl.batch, wl.n_visual)) / 8.0).astype(np.float32)
    # Region (1, 0), budget 300: the 300-th largest score IS zero.  90 positive scores and 30 positive denormals
    # rank first; the other 180 kept tokens are zeros of either sign, which compare equal as floats, so the lowest
    # indices among them win whatever their sign; negative denormals and negative scores rank below every zero.
    z = np.where(rng.integers(0, 2, size=wl.n_visual) == 1, np.float32(-0.0), np.float32(0.0)).astype(np.float32)
    where = rng.permutation(wl.n_visual)
    z[where[:90]] = 0.5
    z[where[90:120]] = 1e-42
    z[where[120:150]] = -1e-42
    z[where[150:200]] = -0.25
    z[:5] = [-0.0, 0.0, 1e-42, 1e-42, -0.0]
    scores[1, 0] = z
    n_pos, n_zero = int((z > 0).sum()), int((z == 0).sum())
    assert n_pos < 300 < n_pos + n_zero and np.signbit(z[z == 0]).any() and not np.signbit(z[z == 0]).all()
    # a layer that keeps nothing, one that keeps one token, two that keep everything; both sequences sum to T
    budgets = np.array([[0, 200], [300, wl.n_visual], [1, 100], [wl.n_visual, 1]], np.int32)
    T = int(budgets[:, 0].sum())
    assert T == int(budgets[:, 1].sum())
    ratio = T / (wl.n_visual * wl.n_layers)
    dm = oracle_dims(oracle, wl)
    assert oracle.total_kept(wl.n_visual, wl.n_layers, ratio) == T
    k_hm = k.permute(0, 1, 3, 2, 4).contiguous()    # head-major storage [L,B,Hkv,N,d]
    v_hm = v.permute(0, 1, 3, 2, 4).contiguous()
    cp = oracle.compact(dm, 2, u16(k_hm), u16(v_hm), scores, budgets)
    gp = GpuPath(wl, ratio=ratio, device=DEV, slack=2)
    gp.set_full(k_hm.to(DEV), v_hm.to(DEV))
    sc_d, bud_d = torch.from_numpy(scores).to(DEV), torch.from_numpy(budgets).to(DEV)
    # offsets/lens for these hand-made budgets: written here the way aircache_budget lays regions out
    sizes = budgets.reshape(-1).astype(np.int64) + wl.n_text + 2
    gp.offsets.copy_(torch.from_numpy(np.concatenate([[0], np.cumsum(sizes)])))
    gp.lens.copy_(torch.from_numpy((budgets.reshape(-1) + wl.n_text).astype(np.int32)))
    gp.compact(scores=sc_d, budgets=bud_d)
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)
    # the same through the workspace-held index list
    gp.k_c.zero_(); gp.v_c.zero_()
    gp.compact(scores=sc_d, budgets=bud_d, want_kept=False)
    compare_cache(gp, cp)


@pytest.mark.parametrize("case", list(CASES))
def test_decode_parity_on_oracle_cache(oracle, case):
    wl = CASES[case]
    slack = 4
    ref = oracle_path(oracle, wl, slack=slack)
    cp = ref["compact"]
    gp = make_gpu(wl, ref, slack=slack)
    # poison everything, then upload only the valid rows: slack rows stay NaN and must not leak
    gp.k_c.fill_(float("nan")); gp.v_c.fill_(float("nan"))
    kc = torch.from_numpy(cp["k"].view(np.int16)).view(torch.bfloat16)
    vc = torch.from_numpy(cp["v"].view(np.int16)).view(torch.bfloat16)
    for r in range(len(cp["lens"])):
        a, n = int(cp["offsets"][r]), int(cp["lens"][r])
        gp.k_c[a:a + n] = kc[a:a + n].to(DEV)
        gp.v_c[a:a + n] = vc[a:a + n].to(DEV)
    gp.offsets.copy_(torch.from_numpy(cp["offsets"]))
    gp.lens.copy_(torch.from_numpy(cp["lens"]))
    for step in range(2):
        q = decode_queries(wl, step, "cpu")
        want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q), wl.scale)
        gp.out.fill_(float("nan"))
        gp.decode(q.to(DEV))
        assert gp.status() == 0
        got = gp.out.cpu().numpy()
        assert np.isfinite(got).all()
        err = rel_row_err(got, want)
        assert err <= TOL, err


def test_decode_tiny_and_empty_regions(oracle):
    """Regions of 0, 1, 15, 16, 17 and 33 rows next to long ones."""
    wl = small("tiny", L=2, Hq=28, Hkv=4, d=128, B=4, Nv=400, Nt=8, W=4)
    rng = np.random.default_rng(11)
    lens = np.array([0, 1, 15, 16, 17, 33, 300, 64], np.int32)
    sizes = lens.astype(np.int64) + 3
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    rows = int(offsets[-1])
    from workloads.synth import to_u16
    kc = torch.from_numpy(rng.standard_normal((rows, 4, 128)).astype(np.float32)).to(torch.bfloat16)
    vc = torch.from_numpy(rng.standard_normal((rows, 4, 128)).astype(np.float32)).to(torch.bfloat16)
    q = decode_queries(wl, 0, "cpu")
    dm = oracle_dims(oracle, wl)
    want = oracle.decode(dm, to_u16(kc), to_u16(vc), offsets, lens, u16(q), wl.scale)
    gp = GpuPath(wl, ratio=1.0, device=DEV, slack=3)
    gp.k_c.fill_(float("nan")); gp.v_c.fill_(float("nan"))
    for r in range(len(lens)):
        a, n = int(offsets[r]), int(lens[r])
        gp.k_c[a:a + n] = kc[a:a + n].to(DEV)
        gp.v_c[a:a + n] = vc[a:a + n].to(DEV)
    gp.offsets.copy_(torch.from_numpy(offsets)); gp.lens.copy_(torch.from_numpy(lens))
    gp.out.fill_(float("nan"))
    gp.decode(q.to(DEV))
    assert gp.status() == 0
    got = gp.out.cpu().numpy()
    assert np.isfinite(got).all()
    assert (got.reshape(8, -1)[0] == 0).all()            # empty region -> zeros
    assert rel_row_err(got, want) <= TOL


# --------------------------------------------------------------------------------------------------
# end to end: CUDA stages chained, against the chained oracle
# --------------------------------------------------------------------------------------------------
def run_chain(gp, ref):
    gp.score(ref["qw"].to(DEV), alpha=ref["alpha"])
    gp.budget()
    gp.compact()


@pytest.mark.parametrize("case", ["c1", "s7b", "s72b", "kv2", "maxreg", "w128"])
def test_end_to_end_chain(oracle, case):
    wl = CASES[case]
    ref = oracle_path(oracle, wl)
    gp = make_gpu(wl, ref)
    run_chain(gp, ref)
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"])
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
    cp = ref["compact"]
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)
    q = decode_queries(wl, 0, "cpu")
    want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q), wl.scale)
    gp.decode(q.to(DEV))
    assert gp.status() == 0
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL
    # text rows are never evicted and sit after the kept visual rows, in order
    kc = u16(gp.k_c)
    kl = u16(logical(ref["k"]))
    for r in range(len(cp["lens"])):
        l, b = divmod(r, wl.batch)
        a, n = int(cp["offsets"][r]), int(cp["lens"][r])
        text = kl[l, b, :, wl.n_visual:, :].transpose(1, 0, 2)
        assert np.array_equal(kc[a + n - wl.n_text:a + n], text)


def test_full_retention_equals_full_cache_decode(oracle):
    wl = CASES["s7b"]
    ref = oracle_path(oracle, wl, ratio=1.0)
    gp = make_gpu(wl, ref)
    run_chain(gp, ref)
    assert (gp.budgets.cpu().numpy() == wl.n_visual).all()
    q = decode_queries(wl, 0, "cpu")
    # full-cache reference: one region per (l, b) holding every token, straight from the generator output
    L, B, N = wl.n_layers, wl.batch, wl.n_tokens
    kf = u16(ref["k"]).reshape(L * B * N, wl.n_kv_heads, wl.head_dim)
    vf = u16(ref["v"]).reshape(L * B * N, wl.n_kv_heads, wl.head_dim)
    offs = (np.arange(L * B + 1) * N).astype(np.int64)
    lens = np.full(L * B, N, np.int32)
    want = oracle.decode(ref["dims"], kf, vf, offs, lens, u16(q), wl.scale)
    gp.decode(q.to(DEV))
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL


@pytest.mark.parametrize("case,alpha", [("s7b", 0.9), ("s7b", 0.0), ("c1", 0.9), ("many", 0.9)])
def test_scoring_layer_by_layer_equals_one_call(oracle, case, alpha):
    """Algorithm 1's first loop taken a layer (or a few layers) at a time: aircache_score_layers over any split of
    the layers gives the same elite sets and, up to the rounding of a different chunking of the keys, the same
    scores as one aircache_score call; both match the oracle; equal calls give equal bits."""
    import paper_2503_23956_b200 as ac
    wl = CASES[case]
    ref = oracle_path(oracle, wl, alpha=alpha)
    gp = make_gpu(wl, ref)
    qw = ref["qw"].to(DEV)
    gp.score(qw, alpha=alpha)
    whole, whole_mask = gp.scores.clone(), gp.mask.clone()
    L = wl.n_layers
    for ranges in ([(l, 1) for l in range(L)], [(0, L // 2), (L // 2, L - L // 2)][::-1]):
        gp.scores.fill_(float("nan")); gp.mask.fill_(-1)
        for begin, count in ranges:
            ac.aircache_score_layers(gp.sh, gp.full, qw, alpha, begin, count, gp.scores, gp.mask, gp.ws)
        assert gp.status() == 0
        assert torch.equal(gp.mask, whole_mask)
        assert rel_elem_err(gp.scores.cpu().numpy(), whole.cpu().numpy()) <= 1e-5
        assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL
    # a single layer leaves the other layers' rows alone, and the same call twice gives the same bits
    gp.scores.fill_(float("nan"))
    ac.aircache_score_layers(gp.sh, gp.full, qw, alpha, L - 1, 1, gp.scores, gp.mask, gp.ws)
    assert torch.isnan(gp.scores[:L - 1]).all()
    last = gp.scores[L - 1].clone()
    assert rel_elem_err(last.cpu().numpy(), whole[L - 1].cpu().numpy()) <= 1e-5
    ac.aircache_score_layers(gp.sh, gp.full, qw, alpha, L - 1, 1, gp.scores, gp.mask, gp.ws)
    assert torch.equal(gp.scores[L - 1], last)
    assert np.array_equal(whole_mask.cpu().numpy().view(np.uint64), ref["mask"])
    assert rel_elem_err(whole.cpu().numpy(), ref["scores"]) <= TOL


def test_system_prompt_prefix_as_leading_text_rows(oracle):
    """A system prompt handed over as the leading text rows: it lies outside the last W text rows that Eq. 5 draws
    its candidates from and outside the softmax of Eq. 7, so the scores, budgets and kept visual tokens are those of
    the cache without it (however loud its keys), every prefix row is in the compressed cache, and decode attends
    to it like the oracle does."""
    wl = CASES["s7b"]
    P = 24
    ref = oracle_path(oracle, wl)
    rng = np.random.default_rng(31)
    Nv = wl.n_visual
    shape = (wl.n_layers, wl.batch, P, wl.n_kv_heads, wl.head_dim)
    pk = torch.from_numpy((rng.standard_normal(shape) * 30.0).astype(np.float32)).to(torch.bfloat16)
    pv = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    k2 = torch.cat([ref["k"][:, :, :Nv], pk, ref["k"][:, :, Nv:]], dim=2).contiguous()     # token-major storage
    v2 = torch.cat([ref["v"][:, :, :Nv], pv, ref["v"][:, :, Nv:]], dim=2).contiguous()
    wl2 = wl.with_(name="s7b_sys", n_text=wl.n_text + P)
    gp = GpuPath(wl2, ratio=ref["ratio"], device=DEV)
    gp.set_full(logical(k2.to(DEV)), logical(v2.to(DEV)))
    gp.score(ref["qw"].to(DEV), alpha=ref["alpha"])
    gp.budget()
    gp.compact()
    assert gp.status() == 0
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"])
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
    assert np.array_equal(gp.kept.cpu().numpy()[:len(ref["compact"]["kept_idx"])], ref["compact"]["kept_idx"])
    dm2 = oracle_dims(oracle, wl2)
    cp2 = oracle.compact(dm2, 0, u16(logical(k2)), u16(logical(v2)), ref["scores"], ref["budgets"])
    compare_cache(gp, cp2)
    kc = u16(gp.k_c)
    for r in range(len(cp2["lens"])):
        l, b = divmod(r, wl.batch)
        first_text = int(cp2["offsets"][r]) + int(ref["budgets"][l, b])
        assert np.array_equal(kc[first_text:first_text + P], u16(pk[l, b]))
    q = decode_queries(wl, 0, "cpu")
    want = oracle.decode(dm2, cp2["k"], cp2["v"], cp2["offsets"], cp2["lens"], u16(q), wl.scale)
    gp.decode(q.to(DEV))
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL


@pytest.mark.parametrize("case,alpha", [("s7b", 0.9), ("s72b", 0.9), ("c1", 0.9), ("kv2", 0.0), ("mha64", 0.9), ("g16", 0.9)])
def test_per_kv_head_budgets_whole_chain(oracle, case, alpha):
    """Per-KV-head mode: Eq. 8 averaged over a KV group's heads, Eq. 9-11 over the (layer, KV head) cells of a
    sequence, every cell's own top-k and stretch of the ragged cache, decode and the fused append - against the
    per-KV-group oracle.  Integer results equal, scores and outputs within 2e-3."""
    import paper_2503_23956_b200 as ac
    wl = CASES[case]
    slack = 2
    k, v, qw = cpu_inputs(wl)
    dm = oracle_dims(oracle, wl)
    kl, vl = u16(logical(k)), u16(logical(v))
    sc = oracle.score_groups(dm, kl, u16(qw), wl.scale, alpha)
    st, sk = oracle.moments(sc["scores"])
    bud = oracle.allocate_groups(st, sk, wl.n_visual, wl.ratio)
    cp = oracle.compact_groups(dm, slack, kl, vl, sc["scores"], bud)
    assert (bud.sum(axis=(0, 2)) == oracle.total_kept(wl.n_visual, wl.n_layers * wl.n_kv_heads, wl.ratio)).all()

    gp = GpuPath(wl, device=DEV, slack=slack, per_kv_head=1)
    gp.set_full(logical(k.to(DEV)), logical(v.to(DEV)))
    gp.score(qw.to(DEV), alpha=alpha)
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), sc["elite_mask"])
    assert rel_elem_err(gp.scores.cpu().numpy(), sc["scores"]) <= TOL
    # integer stages on the oracle's score bits, then the chained CUDA path
    sc_d = torch.from_numpy(sc["scores"]).to(DEV)
    gp.budget(scores=sc_d)
    assert np.array_equal(gp.budgets.cpu().numpy(), bud)
    assert np.allclose(gp.strength.cpu().numpy(), st, rtol=1e-12, atol=0)
    assert np.allclose(gp.skew.cpu().numpy(), sk, rtol=1e-9, atol=1e-12)
    gp.compact(scores=sc_d)
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)
    gp.k_c.fill_(float("nan")); gp.v_c.fill_(float("nan"))
    gp.budget()
    gp.compact()
    assert gp.status() == 0
    assert np.array_equal(gp.budgets.cpu().numpy(), bud)
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)
    # decode: every query head attends to the cell of its KV head
    gdm = oracle.group_decode_dims(dm)
    cells, G = wl.n_layers * wl.batch * wl.n_kv_heads, wl.group
    q = decode_queries(wl, 0, "cpu")
    want = oracle.decode(gdm, cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q).reshape(cells, 1, G, wl.head_dim),
                         wl.scale).reshape(q.shape)
    gp.out.fill_(float("nan"))
    gp.decode(q.to(DEV))
    assert gp.status() == 0
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL
    # Eq. 2 fused: one new row per cell
    rng = np.random.default_rng(3)
    kn = torch.from_numpy(rng.standard_normal((cells, 1, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
    vn = torch.from_numpy(rng.standard_normal((cells, 1, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
    k_o, v_o, lens = cp["k"].copy(), cp["v"].copy(), cp["lens"].copy()
    for c in range(cells):
        k_o[cp["offsets"][c] + lens[c]] = u16(kn)[c]
        v_o[cp["offsets"][c] + lens[c]] = u16(vn)[c]
    lens += 1
    q1 = decode_queries(wl, 1, "cpu")
    want = oracle.decode(gdm, k_o, v_o, cp["offsets"], lens, u16(q1).reshape(cells, 1, G, wl.head_dim),
                         wl.scale).reshape(q1.shape)
    ac.aircache_decode_step(gp.sh, gp.cache, q1.to(DEV), kn.to(DEV), vn.to(DEV), 0, gp.out, gp.ws)
    assert gp.status() == 0
    assert np.array_equal(gp.lens.cpu().numpy(), lens)
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL
    ac.aircache_append(gp.sh, gp.cache, kn.to(DEV), vn.to(DEV), 1)
    assert np.array_equal(gp.lens.cpu().numpy(), lens + 1)


def test_per_kv_head_with_one_kv_head_is_the_per_layer_method(oracle):
    """With a single KV head the cells are the regions: the flag changes nothing, bit for bit."""
    wl = CASES["kv1"]
    ref = oracle_path(oracle, wl)
    outs = []
    for flag in (0, 1):
        gp = GpuPath(wl, device=DEV, per_kv_head=flag)
        gp.set_full(logical(ref["k"].to(DEV)), logical(ref["v"].to(DEV)))
        run_chain(gp, ref)
        gp.decode(decode_queries(wl, 0, DEV))
        outs.append([t.cpu().numpy().reshape(-1).copy()
                     for t in (gp.scores, gp.budgets, gp.kept, gp.k_c.view(torch.int16), gp.out)])
    for a, b in zip(*outs):
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8))
    assert np.array_equal(outs[0][1].reshape(ref["budgets"].shape), ref["budgets"])


def test_results_are_bit_reproducible(oracle):
    wl = CASES["s7b"]
    ref = oracle_path(oracle, wl)
    outs = []
    for _ in range(2):
        gp = make_gpu(wl, ref)
        run_chain(gp, ref)
        q = decode_queries(wl, 1, DEV)
        gp.decode(q)
        outs.append((gp.scores.cpu().numpy().copy(), gp.budgets.cpu().numpy().copy(),
                     gp.kept.cpu().numpy().copy(), gp.out.cpu().numpy().copy()))
    for a, b in zip(*outs):
        assert np.array_equal(a, b)


def test_append_then_decode(oracle):
    """Eq. 2: three appended tokens per region land in the slack rows and take part in the next step."""
    wl = CASES["s7b"]
    slack = 3
    ref = oracle_path(oracle, wl, slack=slack)
    cp = ref["compact"]
    gp = make_gpu(wl, ref, slack=slack)
    run_chain(gp, ref)
    import paper_2503_23956_b200 as ac
    rng = np.random.default_rng(5)
    k_o, v_o, lens = cp["k"].copy(), cp["v"].copy(), cp["lens"].copy()
    LB = wl.n_layers * wl.batch
    for i in range(slack):
        kn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        vn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        ac.aircache_append(gp.sh, gp.cache, kn.to(DEV), vn.to(DEV), i)
        for r in range(LB):
            k_o[cp["offsets"][r] + lens[r]] = u16(kn)[r]
            v_o[cp["offsets"][r] + lens[r]] = u16(vn)[r]
        lens += 1
    assert ac.aircache_append(gp.sh, gp.cache, kn.to(DEV), vn.to(DEV), slack, check=False) == ac.ERR_CAPACITY
    assert np.array_equal(gp.lens.cpu().numpy(), lens)
    q = decode_queries(wl, 0, "cpu")
    want = oracle.decode(ref["dims"], k_o, v_o, cp["offsets"], lens, u16(q), wl.scale)
    gp.decode(q.to(DEV))
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL


@pytest.mark.parametrize("case", ["s7b", "c1", "s72b", "kv1long", "many"])
def test_fused_decode_step_appends_and_attends(oracle, case):
    """aircache_decode_step: the new token's K/V land in the slack rows, take part in the same call's attention,
    and lens grows - checked against the oracle on the cache extended by hand, three steps in a row."""
    import paper_2503_23956_b200 as ac
    wl = CASES[case]
    slack = 3
    ref = oracle_path(oracle, wl, slack=slack)
    cp = ref["compact"]
    gp = make_gpu(wl, ref, slack=slack)
    run_chain(gp, ref)
    rng = np.random.default_rng(17)
    k_o, v_o, lens = cp["k"].copy(), cp["v"].copy(), cp["lens"].copy()
    LB = wl.n_layers * wl.batch
    for i in range(slack):
        kn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        vn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        for r in range(LB):
            k_o[cp["offsets"][r] + lens[r]] = u16(kn)[r]
            v_o[cp["offsets"][r] + lens[r]] = u16(vn)[r]
        lens += 1
        q = decode_queries(wl, i, "cpu")
        want = oracle.decode(ref["dims"], k_o, v_o, cp["offsets"], lens, u16(q), wl.scale)
        gp.out.fill_(float("nan"))
        ac.aircache_decode_step(gp.sh, gp.cache, q.to(DEV), kn.to(DEV), vn.to(DEV), i, gp.out, gp.ws)
        assert gp.status() == 0
        assert np.array_equal(gp.lens.cpu().numpy(), lens)
        assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL
    # the appended rows are in the cache, bit for bit
    kc, vc = u16(gp.k_c), u16(gp.v_c)
    for r in range(LB):
        a, n = int(cp["offsets"][r]), int(lens[r])
        assert np.array_equal(kc[a:a + n], k_o[a:a + n]) and np.array_equal(vc[a:a + n], v_o[a:a + n])
    assert ac.aircache_decode_step(gp.sh, gp.cache, q.to(DEV), kn.to(DEV), vn.to(DEV), slack, gp.out, gp.ws,
                                   check=False) == ac.ERR_CAPACITY


@pytest.mark.parametrize("case", ["s7b", "s72b", "kv2"])
def test_decode_plan_kept_between_calls(oracle, case):
    """Head-split launches keep their plan in the workspace and reuse it while the regions' unit counts stay the
    same.  The rows in use must still be read afresh: a region one row shorter (same unit count, plan reused), a
    region cut to a few rows (other unit count, plan redone) and the original lengths again, all on one workspace."""
    wl = CASES[case]
    ref = oracle_path(oracle, wl)
    cp = ref["compact"]
    gp = make_gpu(wl, ref)
    run_chain(gp, ref)
    q = decode_queries(wl, 0, "cpu")
    qd = q.to(DEV)

    def both(lens):
        gp.lens.copy_(torch.from_numpy(lens).to(DEV))
        want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], lens, u16(q), wl.scale)
        gp.out.fill_(float("nan"))
        gp.decode(qd)
        assert gp.status() == 0
        got = gp.out.cpu().numpy().copy()
        assert rel_row_err(got, want) <= TOL
        return got

    lens0 = cp["lens"].copy()
    first = both(lens0)
    again = both(lens0)                     # the kept plan
    assert np.array_equal(first, again)
    lens1 = lens0.copy()
    lens1[1] -= 1                           # same units (unless the length was 1 mod the unit): fresh row count
    both(lens1)
    lens2 = lens1.copy()
    lens2[0] = 5                            # one unit instead of several
    lens2[-1] = max(1, lens2[-1] // 2)
    both(lens2)
    both(lens2)
    back = both(lens0)
    assert np.array_equal(first, back)


def test_one_workspace_serves_different_caches_in_turn(oracle):
    """The plans a decode launch keeps in the workspace belong to the unit counts it saw: two caches of the same
    shape but different retention ratios (other lengths, other unit counts) decode alternately through ONE
    workspace, and every result is the one the cache gets with a workspace of its own."""
    import paper_2503_23956_b200 as ac
    wl = CASES["s7b"]
    refs = [oracle_path(oracle, wl, ratio=0.1), oracle_path(oracle, wl, ratio=0.6)]
    paths = [make_gpu(wl, ref) for ref in refs]
    for gp, ref in zip(paths, refs):
        run_chain(gp, ref)
    q = decode_queries(wl, 0, "cpu")
    qd = q.to(DEV)
    wants = [oracle.decode(ref["dims"], ref["compact"]["k"], ref["compact"]["v"], ref["compact"]["offsets"],
                           ref["compact"]["lens"], u16(q), wl.scale) for ref in refs]
    own = []
    for gp in paths:
        gp.decode(qd)
        own.append(gp.out.cpu().numpy().copy())
    shared_ws = paths[0].ws
    for turn in range(6):
        i = turn % 2 if turn < 4 else 1          # A B A B B B: misses, then hits
        gp = paths[i]
        gp.out.fill_(float("nan"))
        ac.aircache_decode_attn(gp.sh, gp.cache, qd, gp.out, shared_ws)
        assert ac.aircache_check_status(shared_ws, check=False) == 0
        got = gp.out.cpu().numpy()
        assert np.array_equal(got, own[i])
        assert rel_row_err(got, wants[i]) <= TOL


@pytest.mark.parametrize("slack", [0, 2])
def test_sequences_of_different_lengths_share_one_cache(oracle, slack):
    """Requests whose sequences differ in N_v and N_t are compressed by separate calls into ONE pair of K'/V'
    buffers (first_row, stretches of shared offsets / lens arrays); a single decode launch then attends over the
    regions of all of them.  Every request's budgets, kept rows and outputs equal the oracle run on it alone."""
    import paper_2503_23956_b200 as ac
    seqs = [small("ragA", L=3, B=1, Nv=1000, Nt=40), small("ragB", L=3, B=1, Nv=515, Nt=64, W=9),
            small("ragC", L=3, B=1, Nv=300, Nt=20, W=8, ratio=0.33)]
    refs = [oracle_path(oracle, wl, slack=slack) for wl in seqs]
    paths = [GpuPath(wl, ratio=ref["ratio"], device=DEV, slack=slack) for wl, ref in zip(seqs, refs)]
    rows = [ac.aircache_total_rows(gp.sh, ref["ratio"]) for gp, ref in zip(paths, refs)]
    regions = [wl.n_layers * wl.batch for wl in seqs]
    total, n_reg = sum(rows), sum(regions)
    wl0 = seqs[0]
    k_c = torch.zeros((total, wl0.n_kv_heads, wl0.head_dim), dtype=torch.bfloat16, device=DEV)
    v_c = torch.zeros_like(k_c)
    offsets = torch.full((n_reg + 1,), -1, dtype=torch.int64, device=DEV)
    lens = torch.full((n_reg,), -1, dtype=torch.int32, device=DEV)
    first_row = first_reg = 0
    for gp, ref, n_rows, n_r in zip(paths, refs, rows, regions):
        gp.set_full(logical(ref["k"].to(DEV)), logical(ref["v"].to(DEV)))
        gp.cache = ac.ragged_view(k_c, v_c, offsets.data_ptr() + 8 * first_reg, lens.data_ptr() + 4 * first_reg, total,
                                  first_row)
        run_chain(gp, ref)
        assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
        cp = ref["compact"]
        assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
        assert np.array_equal(offsets[first_reg:first_reg + n_r + 1].cpu().numpy(), cp["offsets"] + first_row)
        assert np.array_equal(lens[first_reg:first_reg + n_r].cpu().numpy(), cp["lens"])
        kc, vc = u16(k_c), u16(v_c)
        for r in range(n_r):
            a, n = int(cp["offsets"][r]), int(cp["lens"][r])
            assert np.array_equal(kc[first_row + a:first_row + a + n], cp["k"][a:a + n])
            assert np.array_equal(vc[first_row + a:first_row + a + n], cp["v"][a:a + n])
        first_row += n_rows
        first_reg += n_r
    assert int(offsets[-1].item()) == total
    # one launch over all regions: a shape with as many "layers" as there are regions, batch 1
    sh_all = shape_of(wl0, n_layers=n_reg, batch=1, slack=slack)
    cache_all = ac.ragged_view(k_c, v_c, offsets, lens, total)
    qs = [decode_queries(wl, 0, "cpu") for wl in seqs]
    q_all = torch.cat([q.reshape(-1, wl0.n_q_heads, wl0.head_dim) for q in qs]).contiguous().to(DEV)
    out = torch.full((n_reg, wl0.n_q_heads, wl0.head_dim), float("nan"), dtype=torch.float32, device=DEV)
    ws = torch.empty(ac.aircache_workspace_bytes(sh_all), dtype=torch.uint8, device=DEV)
    ac.aircache_reset_status(ws)
    ac.aircache_decode_attn(sh_all, cache_all, q_all, out, ws)
    assert ac.aircache_check_status(ws, check=False) == 0
    got = out.cpu().numpy()
    first_reg = 0
    for wl, ref, q, n_r in zip(seqs, refs, qs, regions):
        cp = ref["compact"]
        want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q), wl.scale)
        assert rel_row_err(got[first_reg:first_reg + n_r], want) <= TOL
        first_reg += n_r


def _random_workload(seed):
    rng = np.random.default_rng(1000 + seed)
    hkv = int(rng.choice([1, 2, 4, 8]))
    g = int(rng.choice([1, 2, 3, 4, 7, 8, 12, 16]))
    d = int(rng.choice([64, 128]))
    L = int(rng.integers(1, 6))
    B = int(rng.integers(1, 4))
    nv = int(rng.choice([3, 4, 7, 15, 16, 17, 31, 33, 64, 100, 129, 255, 300, 513, 700]))
    nt = int(rng.choice([1, 2, 3, 5, 16, 17, 40, 70]))
    W = int(rng.integers(1, min(nt, 64) + 1))
    ratio = float(rng.choice([0.0, 0.05, 0.1, 0.33, 0.5, 0.9, 1.0]))
    alpha = float(rng.choice([0.0, 0.5, 0.9, 0.99, 1.0]))
    slack = int(rng.choice([0, 1, 2, 5]))
    return small(f"rnd{seed}", L=L, Hq=hkv * g, Hkv=hkv, d=d, B=B, Nv=nv, Nt=nt, W=W, ratio=ratio, alpha=alpha), slack


@pytest.mark.parametrize("seed", range(32))
def test_random_shapes_whole_chain(oracle, seed):
    """Seeded random shapes (head layouts, head_dim, tiny and ragged token counts, window sizes, retention 0..1,
    thresholds 0..1, slack): the whole chain, one decode and - when there is slack - one fused decode step."""
    import paper_2503_23956_b200 as ac
    wl, slack = _random_workload(seed)
    ref = oracle_path(oracle, wl, slack=slack)
    cp = ref["compact"]
    gp = make_gpu(wl, ref, slack=slack)
    run_chain(gp, ref)
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"]), wl
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL, wl
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"]), wl
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"]), wl
    compare_cache(gp, cp)
    q = decode_queries(wl, 0, "cpu")
    want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q), wl.scale)
    gp.out.fill_(float("nan"))
    gp.decode(q.to(DEV))
    assert gp.status() == 0
    assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL, wl
    if slack > 0:
        rng = np.random.default_rng(seed)
        LB = wl.n_layers * wl.batch
        kn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        vn = torch.from_numpy(rng.standard_normal((LB, wl.n_kv_heads, wl.head_dim)).astype(np.float32)).to(torch.bfloat16)
        k_o, v_o, lens = cp["k"].copy(), cp["v"].copy(), cp["lens"].copy()
        for r in range(LB):
            k_o[cp["offsets"][r] + lens[r]] = u16(kn)[r]
            v_o[cp["offsets"][r] + lens[r]] = u16(vn)[r]
        lens += 1
        q1 = decode_queries(wl, 1, "cpu")
        want = oracle.decode(ref["dims"], k_o, v_o, cp["offsets"], lens, u16(q1), wl.scale)
        ac.aircache_decode_step(gp.sh, gp.cache, q1.to(DEV), kn.to(DEV), vn.to(DEV), 0, gp.out, gp.ws)
        assert gp.status() == 0
        assert np.array_equal(gp.lens.cpu().numpy(), lens)
        assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL, wl


def test_bounded_wait_ends_in_an_error_code_not_a_hang():
    """A wait that nothing satisfies gives up after its poll limit: the kernel returns, the status word is set,
    aircache_check_status reports the timeout, a reset clears it and the workspace is usable again."""
    import time
    import paper_2503_23956_b200 as ac
    wl = CASES["c1"]
    gp = GpuPath(wl, device=DEV)
    assert gp.status() == 0
    t0 = time.time()
    ac.aircache_selftest_wait_timeout(gp.ws)
    assert gp.status() == ac.ERR_TIMEOUT
    assert time.time() - t0 < 20.0
    ac.aircache_reset_status(gp.ws)
    assert gp.status() == 0
    # the context is intact: a normal decode still works afterwards
    k, v, qw = gen_inputs(wl, DEV)
    gp.set_full(logical(k), logical(v))
    gp.score(qw); gp.budget(); gp.compact()
    gp.decode(decode_queries(wl, 0, DEV))
    assert gp.status() == 0 and torch.isfinite(gp.out).all()


@pytest.mark.parametrize("damage", ["budgets_too_large", "offsets_beyond_the_buffers", "offsets_negative"])
def test_compaction_reports_budgets_and_offsets_that_do_not_fit(oracle, damage):
    """aircache_compact reads budgets and offsets from device memory.  When a caller has written values there
    that do not fit the buffers, the rows and list entries concerned are left unwritten, nothing outside the
    buffers is touched (guard rows behind K', V' and the kept list stay as they were), aircache_check_status
    reports AIRCACHE_ERR_INCONSISTENT, and after a reset the same buffers serve a correct run."""
    import paper_2503_23956_b200 as ac
    wl = CASES["s7b"]
    ref = oracle_path(oracle, wl)
    gp = make_gpu(wl, ref)
    guard = 64
    gp.k_c = torch.full((gp.rows + guard,) + tuple(gp.k_c.shape[1:]), 1.5, dtype=torch.bfloat16, device=DEV)
    gp.v_c = torch.full_like(gp.k_c, 2.5)
    gp.kept = torch.full((gp.kept_n + guard,), -7, dtype=torch.int32, device=DEV)
    gp.cache = ac.ragged_view(gp.k_c, gp.v_c, gp.offsets, gp.lens, gp.rows)
    gp.score(ref["qw"].to(DEV))
    gp.budget()
    assert gp.status() == 0
    if damage == "budgets_too_large":
        gp.budgets.fill_(wl.n_visual)
    elif damage == "offsets_beyond_the_buffers":
        gp.offsets[1:] += 1 << 40
    else:
        gp.offsets[1:] -= 1 << 40
    gp.compact()
    assert gp.status() == ac.ERR_INCONSISTENT
    assert ac.aircache_strerror(ac.ERR_INCONSISTENT) != ac.aircache_strerror(-12345)
    assert (gp.k_c[gp.rows:] == 1.5).all() and (gp.v_c[gp.rows:] == 2.5).all()
    assert (gp.kept[gp.kept_n:] == -7).all()
    ac.aircache_reset_status(gp.ws)
    gp.budget()
    gp.compact()
    assert gp.status() == 0
    compare_cache(gp, ref["compact"])
    assert (gp.k_c[gp.rows:] == 1.5).all() and (gp.kept[gp.kept_n:] == -7).all()


@pytest.mark.parametrize("pinned_v", [True, False])
def test_pipeline_host_matches_staged_calls(oracle, pinned_v):
    """Host inputs in, host outputs out, equal to the staged calls bit for bit - with V in page-locked memory
    (compaction reads the surviving rows from it in place; the device buffer for V is poisoned and stays so) and
    with V in pageable memory (uploaded whole)."""
    import paper_2503_23956_b200 as ac
    wl = CASES["c1"]
    ref = oracle_path(oracle, wl)
    gp = make_gpu(wl, ref)
    run_chain(gp, ref)
    n_steps = 3
    q_steps = torch.stack([decode_queries(wl, s, "cpu") for s in range(n_steps)]).contiguous()
    staged = []
    for s in range(n_steps):
        gp.decode(q_steps[s].to(DEV))
        staged.append(gp.out.cpu().numpy().copy())
    gp2 = GpuPath(wl, ratio=ref["ratio"], device=DEV)
    h_k = ref["k"].contiguous().pin_memory()
    h_v = ref["v"].contiguous().pin_memory() if pinned_v else ref["v"].contiguous().clone()
    assert ac.aircache_host_range_is_mapped(h_v) == pinned_v
    h_full = ac.full_view(logical(h_k), logical(h_v))
    d_k = torch.empty_like(h_k, device=DEV)
    d_v = torch.full(h_v.shape, float("nan"), dtype=h_v.dtype, device=DEV)
    h_qw = ref["qw"].contiguous().pin_memory()
    d_qw = torch.empty_like(h_qw, device=DEV)
    h_q = q_steps.pin_memory()
    d_q = torch.empty_like(h_q, device=DEV)
    d_out = torch.empty((n_steps,) + tuple(gp.out.shape), dtype=torch.float32, device=DEV)
    h_out = torch.empty(d_out.shape, dtype=torch.float32).pin_memory()
    h_bud = torch.empty(gp.budgets.shape, dtype=torch.int32).pin_memory()
    ac.aircache_pipeline_host(gp2.sh, h_full, h_k.numel(), d_k, d_v, h_qw, d_qw, h_q, d_q, n_steps, wl.alpha,
                              ref["ratio"], 0, gp2.scores, gp2.budgets, gp2.cache, d_out, h_out, h_bud, gp2.ws)
    assert np.array_equal(h_bud.numpy(), ref["budgets"])
    for s in range(n_steps):
        assert np.array_equal(h_out[s].numpy(), staged[s])
    assert bool(torch.isnan(d_v.float()).all()) == pinned_v   # V uploaded only when it could not be read in place


# --------------------------------------------------------------------------------------------------
# full-size configurations, in the launch configuration the benchmark times
# --------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("ratio", [0.10, 0.50, 0.25, 0.05])
def test_config2_full_size(oracle, ratio):
    """Qwen2-7B-shaped single image (28 layers, 7290 + 128 tokens): the whole chain against the whole oracle."""
    wl = CONFIGS["c2"]
    ref = oracle_path(oracle, wl, ratio=ratio)
    gp = make_gpu(wl, ref)
    run_chain(gp, ref)
    assert np.array_equal(gp.mask.cpu().numpy().view(np.uint64), ref["mask"])
    assert rel_elem_err(gp.scores.cpu().numpy(), ref["scores"]) <= TOL
    assert np.array_equal(gp.budgets.cpu().numpy(), ref["budgets"])
    cp = ref["compact"]
    assert np.array_equal(gp.kept.cpu().numpy()[:len(cp["kept_idx"])], cp["kept_idx"])
    compare_cache(gp, cp)
    for step in (0, 1):
        q = decode_queries(wl, step, "cpu")
        want = oracle.decode(ref["dims"], cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(q), wl.scale)
        gp.decode(q.to(DEV))
        assert gp.status() == 0
        assert rel_row_err(gp.out.cpu().numpy(), want) <= TOL


@pytest.mark.parametrize("cfg,batch,seqs", [("c3", 1, (0,)), ("c3", 8, (0, 7)), ("c3", 32, (0, 31)), ("c3", 64, (1, 63)),
                                            ("c4", 4, (1,)), ("c5", 8, (5,))])
def test_batched_configs_sampled_sequences(oracle, cfg, batch, seqs):
    """Batched configurations (7B shapes, and the 72B-shaped long-context one at its full 80 layers x 8
    sequences) at full batch on the GPU; the oracle runs whole sequences sampled from the batch (every stage is independent per sequence, so a sequence's regions compare one to one)."""
    from workloads import full_cache, window_queries
    wl = CONFIGS[cfg].with_(batch=batch)
    gp = GpuPath(wl, device=DEV)
    k, v = full_cache(wl, "k", DEV), full_cache(wl, "v", DEV)
    gp.set_full(logical(k), logical(v))
    qw = window_queries(wl, DEV)
    gp.score(qw)
    gp.budget()
    gp.compact()
    q = decode_queries(wl, 0, DEV)
    gp.decode(q)
    assert gp.status() == 0
    offs, lens = gp.offsets.cpu().numpy(), gp.lens.cpu().numpy()
    kc, vc = u16(gp.k_c), u16(gp.v_c)
    out = gp.out.cpu().numpy()
    assert (gp.budgets.sum(dim=0).cpu().numpy() == oracle.total_kept(wl.n_visual, wl.n_layers, wl.ratio)).all()
    for b in seqs:
        w1 = wl.with_(batch=1)
        dm = oracle_dims(oracle, w1)
        kb, vb = full_cache(wl, "k", "cpu", seqs=[b]), full_cache(wl, "v", "cpu", seqs=[b])
        qwb = window_queries(wl, "cpu", seqs=[b])
        sc = oracle.score(dm, u16(logical(kb)), u16(qwb), wl.scale, wl.alpha)
        assert np.array_equal(gp.mask[:, b].cpu().numpy().view(np.uint64), sc["elite_mask"][:, 0])
        assert rel_elem_err(gp.scores[:, b].cpu().numpy(), sc["scores"][:, 0]) <= TOL
        st, sk = oracle.moments(sc["scores"])
        bud = oracle.allocate(st, sk, wl.n_visual, wl.ratio, 0)
        assert np.array_equal(gp.budgets[:, b].cpu().numpy(), bud[:, 0])
        cp = oracle.compact(dm, 0, u16(logical(kb)), u16(logical(vb)), sc["scores"], bud)
        qb = decode_queries(wl, 0, "cpu", seqs=[b])
        want = oracle.decode(dm, cp["k"], cp["v"], cp["offsets"], cp["lens"], u16(qb), wl.scale)
        for l in range(wl.n_layers):
            r = l * wl.batch + b
            a, n = int(offs[r]), int(lens[r])
            a0, n0 = int(cp["offsets"][l]), int(cp["lens"][l])
            assert n == n0
            assert np.array_equal(kc[a:a + n], cp["k"][a0:a0 + n0])
            assert np.array_equal(vc[a:a + n], cp["v"][a0:a0 + n0])
        assert rel_row_err(out[:, b], want[:, 0]) <= TOL
