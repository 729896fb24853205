"""GPU parity: the CUDA library against the CPU oracle on the same seeded inputs, through the
C ABI. Masks must be bit-exact except rows the oracle flags as ties (k-th / (k+1)-th score gap
below 1e-5 relative), which are counted; attention must stay within 2e-2 (bf16) / 1e-4 (fp32)."""
import numpy as np
import pytest
import torch

from helpers import TIE_GAP, check_mask_invariants, compare_masks, oracle_problem, sample_rows
from oracle import stream_oracle as so
from paper_2510_19875_b200 import workloads as wl

pytestmark = pytest.mark.gpu

ATTN_TOL = {"bf16": 2e-2, "f32": 1e-4}


@pytest.fixture(scope="module")
def S():
    from paper_2510_19875_b200 import stream

    assert stream.stream_version() >= 100
    return stream


def run_mask(S, w, *, impl="auto", block_q=None, block_k=None, k_top=None, causal=True, want_scores=False):
    spec = w.spec
    q, k, _ = w.torch_tensors("cuda")
    res = S.build_mask(q, k, block_q=block_q or spec.block, block_k=block_k or spec.block,
                       k_top=k_top or spec.k_top, causal=causal, impl=impl, want_scores=want_scores, row_tiles=True)
    torch.cuda.synchronize()
    return res


def assert_mask_parity(S, w, rows, *, impl="auto", score_cache=True, **kw):
    spec = w.spec
    res = run_mask(S, w, impl=impl, want_scores=True, **kw)
    mask = res.mask.cpu().numpy()
    st = res.stats()
    assert st.error == 0, f"device error {st.error} (info {st.error_info:#x})"
    check_mask_invariants(mask, spec, block_q=kw.get("block_q"), block_k=kw.get("block_k"), causal=kw.get("causal", True))
    p = oracle_problem(spec, **kw)
    ora = so.build_mask_rows(p, w.q, w.k, rows, score_cache=score_cache, want_scores=True)
    flat = mask.reshape(-1, mask.shape[-1])
    got = flat if rows is None else flat[rows]
    report = compare_masks(got, ora)
    assert report["bad"] == 0, report
    # scores of kept blocks: fp32 accumulation on the GPU against fp64-then-round in the oracle
    sc = res.scores.cpu().numpy().reshape(-1, mask.shape[-1])
    sc = sc if rows is None else sc[rows]
    same = (got == ora["mask"]).all(axis=1)
    fin = np.isfinite(ora["scores"][same])
    np.testing.assert_allclose(sc[same][fin], ora["scores"][same][fin], rtol=2e-5, atol=2e-5)
    assert (sc[same][~fin] == -np.inf).all()
    assert st.rows == flat.shape[0]
    # tiles scored, row by row: every row that is not a near-tie must have scored exactly the
    # oracle's distinct (row, representative block) tiles; the total is the sum of the rows
    rt = res.row_tiles().cpu().numpy().reshape(-1).astype(np.int64)
    assert int(rt.sum()) == st.tiles_scored
    rt = rt if rows is None else rt[rows]
    agree = same & (ora["min_gap"] >= 1e-5)
    assert (rt[agree] == ora["tiles"][agree]).all()
    return report


def small_spec(**kw):
    base = dict(name="t", seed=5, batch=1, n_q_heads=2, n_kv_heads=1, T=512, d=64, block=32, k_top=4, dtype="f32")
    base.update(kw)
    return wl.WorkloadSpec(**base)


GENERIC_CASES = [
    dict(),                                                        # fp32, two levels
    dict(dtype="bf16", d=128, block=64, T=2048, k_top=8, n_q_heads=4, n_kv_heads=2, sink=True),
    dict(T=1000, k_top=5),                                         # ragged T, odd k
    dict(T=777, d=32, block=16, k_top=3, batch=2),                 # batch, ragged, uneven nodes
    dict(T=512, d=16, block=8, k_top=7, dtype="bf16"),
    dict(T=256, k_top=16),                                         # k > N_k: full mask, no levels
    dict(T=64, block=64, k_top=2),                                 # a single key block
    dict(T=1, block=32, k_top=1, n_q_heads=1),                     # one token
    dict(dtype="bf16", d=256, block=32, T=1500, k_top=4, n_q_heads=4, n_kv_heads=1, sink=True),  # head dim 256
    dict(d=256, block=64, T=700, k_top=3),                         # head dim 256, fp32
    dict(T=4096, d=64, block=32, k_top=1, n_q_heads=1),            # k = 1: pure binary descent
]


@pytest.mark.parametrize("kw", GENERIC_CASES)
def test_mask_generic_small(S, kw):
    w = wl.generate(small_spec(**kw))
    assert_mask_parity(S, w, None, impl="generic", score_cache=False)


def tc_spec(**kw):
    base = dict(name="tc", seed=7, batch=1, n_q_heads=4, n_kv_heads=1, T=4096, d=128, block=64, k_top=8, dtype="bf16", sink=True)
    base.update(kw)
    return wl.WorkloadSpec(**base)


TC_CASES = [
    dict(),                                                   # one kv head, four rows per group, 3 levels
    dict(T=2048, k_top=16, n_q_heads=8, n_kv_heads=2),        # N_k = 2k: a single level
    dict(T=8192, k_top=32, n_q_heads=2, n_kv_heads=2),        # one row per group
    dict(T=5000, k_top=5, n_q_heads=7, n_kv_heads=1),         # ragged T, odd k, groups of 4 + 3 heads
    dict(T=3000, k_top=3, n_q_heads=6, n_kv_heads=2, batch=2, local=True),
    dict(T=16384, k_top=1, n_q_heads=1, n_kv_heads=1),        # k = 1
    dict(T=1024, k_top=32, n_q_heads=4, n_kv_heads=4),        # k > N_k
    dict(T=100, k_top=4, n_q_heads=4, n_kv_heads=2),          # two key blocks, ragged
]


@pytest.mark.parametrize("kw", TC_CASES)
def test_mask_tensor_core_small(S, kw):
    w = wl.generate(tc_spec(**kw))
    assert_mask_parity(S, w, None, impl="tensor", score_cache=False)


def test_mask_tensor_core_non_causal(S):
    w = wl.generate(tc_spec(T=3000, k_top=6))
    assert_mask_parity(S, w, None, impl="tensor", score_cache=False, causal=False)


def test_consistency_of_the_two_mask_kernels(S):
    """Not a parity test (each kernel is compared with the oracle above): the two CUDA kernels
    against each other, as a cheap cross-check that they count and score the same tiles."""
    w = wl.generate(tc_spec(T=8192, k_top=16, n_q_heads=8, n_kv_heads=2, anchors=True))
    a = run_mask(S, w, impl="tensor", want_scores=True)
    b = run_mask(S, w, impl="generic", want_scores=True)
    same = (a.mask == b.mask).all(-1)
    assert same.float().mean().item() > 0.97  # the rest are near-ties resolved by rounding
    fin = torch.isfinite(b.scores[same])
    torch.testing.assert_close(a.scores[same][fin], b.scores[same][fin], rtol=2e-5, atol=2e-5)
    assert a.stats().tiles_scored == b.stats().tiles_scored or not same.all()


@pytest.mark.parametrize("bq,bk", [(16, 32), (32, 8), (1, 16), (24, 16)])
def test_mask_generic_unequal_blocks(S, bq, bk):
    w = wl.generate(small_spec(T=700, k_top=5))
    assert_mask_parity(S, w, None, impl="generic", score_cache=False, block_q=bq, block_k=bk)


TOKEN_CASES = [
    dict(T=2048, k_top=4),                                        # 32 key blocks, three levels, 16 groups of 128 tokens
    dict(T=1000, k_top=5, n_q_heads=3, n_kv_heads=1),             # ragged T (last group and last key block partial), odd k
    dict(T=4096, k_top=8, n_q_heads=4, n_kv_heads=2, anchors=True),
    dict(T=3000, k_top=32, n_q_heads=2, n_kv_heads=2),            # k close to N_k: one level
    dict(T=8192, k_top=1, n_q_heads=1, n_kv_heads=1),             # k = 1: binary descent per token
    dict(T=700, k_top=3, batch=2, n_q_heads=2, n_kv_heads=1, local=True),
    dict(T=130, k_top=2),                                         # three key blocks, two groups
]


@pytest.mark.parametrize("kw", TOKEN_CASES)
def test_mask_per_token_tensor_core_small(S, kw):
    """block_q = 1 (every token a row of its own) on the tensor-core path, every row against the oracle."""
    w = wl.generate(tc_spec(**kw))
    assert_mask_parity(S, w, None, impl="tensor", score_cache=False, block_q=1, block_k=64)


def test_mask_per_token_tensor_core_non_causal(S):
    w = wl.generate(tc_spec(T=1500, k_top=6, n_q_heads=2, n_kv_heads=1))
    assert_mask_parity(S, w, None, impl="tensor", score_cache=False, block_q=1, block_k=64, causal=False)


def test_mask_per_token_tensor_core_repeats_and_matches_generic(S):
    w = wl.generate(tc_spec(T=3000, k_top=7, n_q_heads=4, n_kv_heads=2, anchors=True))
    a = run_mask(S, w, impl="tensor", block_q=1, block_k=64, want_scores=True)
    for _ in range(3):
        b = run_mask(S, w, impl="tensor", block_q=1, block_k=64, want_scores=True)
        assert torch.equal(a.mask, b.mask) and torch.equal(a.scores, b.scores)
        assert a.stats().tiles_scored == b.stats().tiles_scored
    c = run_mask(S, w, impl="generic", block_q=1, block_k=64)   # consistency only: both are checked against the oracle
    assert (a.mask == c.mask).all(-1).float().mean().item() > 0.97
    st = a.stats()
    assert st.tile_products >= st.tiles_scored // 64              # every needed tile is inside a computed product


def test_mask_per_token_strided_inputs_and_limits(S):
    """[B, T, H, d] storage through [B, H, T, d] strides gives the same per-token mask (the kernel
    reads Q rows straight from global memory with the caller's strides); shapes the per-token
    tensor-core kernel does not take are refused when it is asked for by name and run on the
    generic kernel otherwise."""
    w = wl.generate(tc_spec(T=1500, k_top=4, n_q_heads=4, n_kv_heads=2))
    q, k, _ = w.torch_tensors("cuda")
    ref = S.build_mask(q, k, block_q=1, block_k=64, k_top=4, impl="tensor")
    assert ref.stats().tile_products > 0
    qs = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    ks = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not qs.is_contiguous()
    got = S.build_mask(qs, ks, block_q=1, block_k=64, k_top=4, impl="tensor")
    assert torch.equal(got.mask, ref.mask)
    # one k per call only: the variable-k build for per-token rows is the generic kernel's
    p = S.make_problem(q, k, block_q=1, block_k=64, k_top=4, impl="tensor")
    k_row = torch.full((1500,), 3, dtype=torch.int32, device="cuda")
    ws = S.new_workspace(p, q.device)
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask_var(p, q, k, k_row, ref.mask.clone(), None, ws, ws.numel())
    assert e.value.status == S.STREAM_ERR_UNSUPPORTED
    var = S.build_mask(q, k, block_q=1, block_k=64, k_top=4, k_row=k_row)   # impl auto: generic kernel
    assert var.stats().tile_products == 0 and ((var.mask >= 0).sum(-1) <= 3).all()
    # block_k other than 64 is not the tensor-core kernel's either
    with pytest.raises(S.StreamError) as e:
        S.build_mask(q, k, block_q=1, block_k=32, k_top=4, impl="tensor")
    assert e.value.status == S.STREAM_ERR_UNSUPPORTED


def test_mask_generic_non_causal(S):
    w = wl.generate(small_spec(T=900, k_top=6, n_q_heads=2, n_kv_heads=2))
    assert_mask_parity(S, w, None, impl="generic", score_cache=False, causal=False)


def test_mask_strided_inputs(S):
    """[B, T, H, d] storage seen through [B, H, T, d] strides gives the same mask."""
    w = wl.generate(small_spec(dtype="bf16", d=128, block=64, T=1024, k_top=4, n_q_heads=4, n_kv_heads=2))
    q, k, _ = w.torch_tensors("cuda")
    ref = S.build_mask(q, k, block_q=64, block_k=64, k_top=4).mask
    qs = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    ks = k.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not qs.is_contiguous()
    for impl in ("generic", "auto"):
        got = S.build_mask(qs, ks, block_q=64, block_k=64, k_top=4, impl=impl).mask
        assert torch.equal(got, ref)


def test_config1_single_head_fp32_all_rows(S):
    w = wl.generate(wl.SPECS["single_head_fp32"])
    rep = assert_mask_parity(S, w, None, score_cache=False)
    assert rep["rows"] == 64


def attention_parity(S, w, rows, *, impl="auto", block_q=None, block_k=None, causal=True, k_top=None):
    """Both sides use the ORACLE's mask, so mask tie exemptions cannot leak into this check."""
    spec = w.spec
    p = oracle_problem(spec, block_q=block_q, block_k=block_k, causal=causal, k_top=k_top)
    bq, bk = p.block_q, p.block_k
    ora_all = so.build_mask_rows(p, w.q, w.k, rows, score_cache=True)
    nqb = so.num_query_blocks(p)
    full = np.full((spec.batch * spec.n_q_heads * nqb, p.k_top), -1, np.int32)
    idx = np.arange(full.shape[0]) if rows is None else rows
    full[idx] = ora_all["mask"]
    q, k, v = w.torch_tensors("cuda")
    mask_dev = torch.from_numpy(full.reshape(spec.batch, spec.n_q_heads, nqb, p.k_top)).cuda()
    out = S.sparse_attention(q, k, v, mask_dev, block_q=bq, block_k=bk, causal=causal, impl=impl)
    torch.cuda.synchronize()
    ref = so.sparse_attention_rows(p, w.q, w.k, w.v, ora_all["mask"], rows)  # [n, bq, d] fp64
    got = out.float().cpu().numpy().reshape(spec.batch * spec.n_q_heads, spec.T, spec.d)
    worst = 0.0
    for i, rid in enumerate(idx):
        bh, qb = divmod(int(rid), nqb)
        lo, hi = qb * bq, min(spec.T, qb * bq + bq)
        worst = max(worst, float(np.abs(got[bh, lo:hi] - ref[i, : hi - lo]).max()))
    assert worst <= ATTN_TOL[spec.dtype], worst
    return worst


@pytest.mark.parametrize("kw", [
    dict(),
    dict(dtype="bf16", d=128, block=64, T=2048, k_top=8, n_q_heads=4, n_kv_heads=2, sink=True),
    dict(T=777, d=32, block=16, k_top=3, batch=2),
    dict(T=256, k_top=16),
    dict(dtype="bf16", d=256, block=32, T=1500, k_top=4, n_q_heads=4, n_kv_heads=1, sink=True),
    dict(d=256, block=64, T=700, k_top=3),
])
def test_attention_generic_small(S, kw):
    w = wl.generate(small_spec(**kw))
    attention_parity(S, w, None, impl="generic")


def test_attention_generic_unequal_blocks_and_non_causal(S):
    w = wl.generate(small_spec(T=700, k_top=5))
    attention_parity(S, w, None, impl="generic", block_q=24, block_k=16)
    attention_parity(S, w, None, impl="generic", causal=False)


ATTN_TC_CASES = [
    dict(),                                                   # two pairs of one kv head
    dict(T=2048, k_top=16, n_q_heads=8, n_kv_heads=2),
    dict(T=5000, k_top=5, n_q_heads=7, n_kv_heads=1),         # ragged T, an odd head left alone in its pair
    dict(T=3000, k_top=3, n_q_heads=6, n_kv_heads=2, batch=2, local=True),
    dict(T=1024, k_top=32, n_q_heads=4, n_kv_heads=4),        # full causal mask, one head per kv head
    dict(T=100, k_top=4, n_q_heads=4, n_kv_heads=2),          # two key blocks, ragged
    dict(T=8192, k_top=32, n_q_heads=8, n_kv_heads=2, anchors=True),
]


@pytest.mark.parametrize("kw", ATTN_TC_CASES)
def test_attention_tensor_core_small(S, kw):
    w = wl.generate(tc_spec(**kw))
    attention_parity(S, w, None, impl="tensor")
    S.stream_check_device_status()


def test_attention_tensor_core_non_causal(S):
    w = wl.generate(tc_spec(T=3000, k_top=6))
    attention_parity(S, w, None, impl="tensor", causal=False)


@pytest.mark.parametrize("causal", [True, False])
# 200: long mask rows leave the tensor-core kernel four ring buffers instead of five
@pytest.mark.parametrize("impl,k_top", [("tensor", 6), ("tensor", 200), ("generic", 6)])
def test_attention_arbitrary_mask(S, impl, causal, k_top):
    """Any int32 mask is legal input: unsorted, with holes, rows of unequal length, blocks after the
    query (all their keys are excluded under a causal C), rows with nothing kept (zeros)."""
    spec = tc_spec(T=2500, k_top=k_top, n_q_heads=6, n_kv_heads=2, batch=2)
    w = wl.generate(spec)
    p = oracle_problem(spec, causal=causal)
    nqb, rng = spec.n_blocks, np.random.default_rng(11)
    mask = rng.integers(0, nqb, size=(spec.n_rows, spec.k_top)).astype(np.int32)
    mask[rng.random(mask.shape) < (0.35 if k_top == 6 else 0.9)] = -1
    mask[rng.random(spec.n_rows) < 0.1] = -1
    q, k, v = w.torch_tensors("cuda")
    mask_dev = torch.from_numpy(mask.reshape(spec.batch, spec.n_q_heads, nqb, spec.k_top)).cuda()
    out = S.sparse_attention(q, k, v, mask_dev, block_q=64, block_k=64, causal=causal, impl=impl)
    torch.cuda.synchronize()
    ref = so.sparse_attention_rows(p, w.q, w.k, w.v, mask, None)
    got = out.float().cpu().numpy().reshape(spec.batch * spec.n_q_heads, spec.T, spec.d)
    for rid in range(spec.n_rows):
        bh, qb = divmod(rid, nqb)
        lo, hi = qb * 64, min(spec.T, qb * 64 + 64)
        assert np.abs(got[bh, lo:hi] - ref[rid, : hi - lo]).max() <= ATTN_TOL["bf16"], rid


def test_full_mask_attention_equals_dense_softmax_attention(S):
    """k covers every causal block: the sparse pass must reproduce dense causal attention."""
    w = wl.generate(small_spec(dtype="bf16", d=128, block=64, T=1024, k_top=16, n_q_heads=4, n_kv_heads=2))
    q, k, v = w.torch_tensors("cuda")
    res = S.build_mask(q, k, block_q=64, block_k=64, k_top=16)
    out = S.sparse_attention(q, k, v, res.mask, block_q=64, block_k=64)
    ref = torch.nn.functional.scaled_dot_product_attention(
        q.double().cpu(), k.double().cpu().repeat_interleave(2, 1), v.double().cpu().repeat_interleave(2, 1), is_causal=True)
    assert (out.double().cpu() - ref).abs().max().item() <= 2e-2


def test_config1_attention(S):
    w = wl.generate(wl.SPECS["single_head_fp32"])
    attention_parity(S, w, None)


def test_run_host_matches_device_calls(S):
    w = wl.generate(small_spec(dtype="bf16", d=128, block=64, T=2048, k_top=8, n_q_heads=4, n_kv_heads=2, sink=True))
    qh, kh, vh = w.torch_tensors("cpu", pin=True)
    q, k, v = qh.cuda(), kh.cuda(), vh.cuda()
    ref = S.build_mask(q, k, block_q=64, block_k=64, k_top=8)
    out_ref = S.sparse_attention(q, k, v, ref.mask, block_q=64, block_k=64)
    p = S.make_problem(qh, kh, block_q=64, block_k=64, k_top=8)
    staging = torch.empty(S.stream_host_staging_bytes(p), dtype=torch.uint8, device="cuda")
    mask_host = torch.empty(ref.mask.shape, dtype=torch.int32).pin_memory()
    out_host = torch.empty(out_ref.shape, dtype=out_ref.dtype).pin_memory()
    S.run_host(qh, kh, vh, mask_host, out_host, staging, block_q=64, block_k=64, k_top=8)
    torch.cuda.synchronize()
    assert torch.equal(mask_host, ref.mask.cpu())
    assert torch.equal(out_host, out_ref.cpu())


def test_run_host_var_matches_device_calls(S):
    """The host path with one k per query block against the device calls it is made of."""
    w = wl.generate(small_spec(dtype="bf16", d=128, block=64, T=4096, k_top=8, n_q_heads=8, n_kv_heads=2, sink=True, batch=2))
    qh, kh, vh = w.torch_tensors("cpu", pin=True)
    q, k, v = qh.cuda(), kh.cuda(), vh.cuda()
    p = S.make_problem(qh, kh, block_q=64, block_k=64, k_top=8)
    k_row = S.k_schedule(p, 0.1)
    assert k_row.min() < k_row.max()
    ref = S.build_mask(q, k, block_q=64, block_k=64, k_top=8, k_row=k_row.cuda())
    out_ref = S.sparse_attention(q, k, v, ref.mask, block_q=64, block_k=64)
    staging = torch.empty(S.stream_host_staging_bytes(p), dtype=torch.uint8, device="cuda")
    mask_host = torch.empty(ref.mask.shape, dtype=torch.int32).pin_memory()
    out_host = torch.empty(out_ref.shape, dtype=out_ref.dtype).pin_memory()
    S.run_host(qh, kh, vh, mask_host, out_host, staging, block_q=64, block_k=64, k_top=8, k_row=k_row)
    torch.cuda.synchronize()
    assert torch.equal(mask_host, ref.mask.cpu())
    assert torch.equal(out_host, out_ref.cpu())
    assert ((mask_host >= 0).sum(-1)[0, 0] == torch.minimum(k_row, torch.arange(1, k_row.numel() + 1, dtype=torch.int32))).all()


@pytest.mark.parametrize("kw", [dict(), dict(T=5000, k_top=5, n_q_heads=7, n_kv_heads=1), dict(T=3000, k_top=3, n_q_heads=6, n_kv_heads=2, batch=2)])
def test_vertical_scores_and_kurtosis(S, kw):
    """Column sums of the GPU mask (binary and score-weighted) and their kurtosis against the oracle
    fed with the same mask and scores."""
    w = wl.generate(tc_spec(**kw))
    spec = w.spec
    res = run_mask(S, w, want_scores=True)
    p = S.make_problem(*w.torch_tensors("cuda")[:2], block_q=spec.block, block_k=spec.block, k_top=spec.k_top)
    op = oracle_problem(spec)
    mask_np = res.mask.cpu().numpy().reshape(-1, spec.k_top)
    sc_np = res.scores.cpu().numpy().reshape(-1, spec.k_top)
    vert, kurt = S.vertical_scores(p, res.mask)
    ref_v, ref_k = so.vertical_scores(op, mask_np)
    assert np.array_equal(vert.cpu().numpy().reshape(ref_v.shape), ref_v)          # counts: exact
    np.testing.assert_allclose(kurt.cpu().numpy().reshape(-1), ref_k, rtol=1e-4)
    wvert, wkurt = S.vertical_scores(p, res.mask, res.scores)
    ref_wv, ref_wk = so.vertical_scores(op, mask_np, sc_np)
    np.testing.assert_allclose(wvert.cpu().numpy().reshape(ref_wv.shape), ref_wv, rtol=1e-5, atol=1e-2)  # fp32 sums of scores ~ 50
    np.testing.assert_allclose(wkurt.cpu().numpy().reshape(-1), ref_wk, rtol=1e-3)


def test_vertical_scores_flags_out_of_range_entries(S):
    w = wl.generate(tc_spec(T=1024, k_top=4))
    q, k, _ = w.torch_tensors("cuda")
    p = S.make_problem(q, k, block_q=64, block_k=64, k_top=4)
    mask = torch.full((1, 4, 16, 4), 16, dtype=torch.int32, device="cuda")  # block 16 does not exist
    with pytest.raises(S.StreamError) as e:
        S.vertical_scores(p, mask)
    assert e.value.status == S.STREAM_ERR_DEVICE_CHECK


def test_mask_difference_of_two_budgets(S):
    """Masks built with k = 6 minus masks built with k = 3 on the same inputs, with the larger
    mask's scores, against the oracle's row-wise difference (integer work: exact)."""
    w = wl.generate(tc_spec(T=3000, n_q_heads=6, n_kv_heads=2, batch=2, local=True))
    big = run_mask(S, w, k_top=6, want_scores=True)
    small = run_mask(S, w, k_top=3)
    diff, dsc = S.mask_difference(big.mask, small.mask, big.scores)
    torch.cuda.synchronize()
    ref, ref_sc = so.mask_difference(big.mask.cpu().numpy().reshape(-1, 6), small.mask.cpu().numpy().reshape(-1, 3),
                                     big.scores.cpu().numpy().reshape(-1, 6))
    assert np.array_equal(diff.cpu().numpy().reshape(-1, 6), ref)
    assert np.array_equal(dsc.cpu().numpy().reshape(-1, 6), ref_sc)
    assert (ref >= 0).any() and (ref[:, 0] < 0).any()  # both non-trivial and empty rows occur
    # wide rows, unsorted, with holes: more than one 32-entry sweep on both sides
    rng = np.random.default_rng(5)
    a = rng.integers(-1, 300, size=(257, 70)).astype(np.int32)
    b = rng.integers(-1, 300, size=(257, 45)).astype(np.int32)
    d2, _ = S.mask_difference(torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda())
    assert np.array_equal(d2.cpu().numpy(), so.mask_difference(a, b)[0])


def variable_k_parity(S, w, k_row, *, impl, attention=True, **kw):
    """Mask rows built with k = k_row[query block] against the oracle's (bit-exact outside ties),
    kept scores, the tile counter, the row counts, and Eq. 2 on the oracle's variable-k mask."""
    spec = w.spec
    p = oracle_problem(spec, **kw)
    bq, bk = p.block_q, p.block_k
    q, k, v = w.torch_tensors("cuda")
    k_dev = torch.from_numpy(k_row).cuda()
    res = S.build_mask(q, k, block_q=bq, block_k=bk, k_top=p.k_top, causal=p.causal, impl=impl, want_scores=True, k_row=k_dev)
    torch.cuda.synchronize()
    st = res.stats()
    assert st.error == 0, f"device error {st.error} (info {st.error_info:#x})"
    mask = res.mask.cpu().numpy().reshape(-1, p.k_top)
    ora = so.build_mask_rows_var(p, w.q, w.k, k_row, want_scores=True)
    report = compare_masks(mask, ora)
    assert report["bad"] == 0, report
    same = (mask == ora["mask"]).all(axis=1)
    sc = res.scores.cpu().numpy().reshape(-1, p.k_top)
    fin = np.isfinite(ora["scores"][same])
    np.testing.assert_allclose(sc[same][fin], ora["scores"][same][fin], rtol=2e-5, atol=2e-5)
    assert (sc[same][~fin] == -np.inf).all()
    # every row holds min(its k, blocks it may look at) entries
    nqb = so.num_query_blocks(p)
    qb = np.arange(mask.shape[0]) % nqb
    last_tok = np.minimum(qb * bq + bq - 1, spec.T - 1) if p.causal else np.full(qb.shape, spec.T - 1)
    want_cnt = np.minimum(np.clip(k_row[qb], 1, p.k_top), last_tok // bk + 1)
    assert ((mask >= 0).sum(1) == want_cnt).all()
    assert st.rows == mask.shape[0]
    if same.all() and (ora["min_gap"] >= 1e-5).all():
        assert st.tiles_scored == int(ora["tiles"].sum())
    if attention:
        mdev = torch.from_numpy(ora["mask"].reshape(spec.batch, spec.n_q_heads, nqb, p.k_top)).cuda()
        out = S.sparse_attention(q, k, v, mdev, block_q=bq, block_k=bk, causal=p.causal, impl=impl)
        torch.cuda.synchronize()
        ref = so.sparse_attention_rows(p, w.q, w.k, w.v, ora["mask"])
        got = out.float().cpu().numpy().reshape(-1, spec.T, spec.d)
        for i in range(mask.shape[0]):
            bh, b_ = divmod(i, nqb)
            lo, hi = b_ * bq, min(spec.T, b_ * bq + bq)
            assert np.abs(got[bh, lo:hi] - ref[i, : hi - lo]).max() <= ATTN_TOL[spec.dtype]
    return report


@pytest.mark.parametrize("impl", ["tensor", "generic"])
@pytest.mark.parametrize("kw,s", [
    (dict(T=5000, k_top=12, n_q_heads=7, n_kv_heads=1), 0.15),    # groups of 4 + 3 heads, ragged T, k from 1 to 12
    (dict(T=8192, k_top=32, n_q_heads=4, n_kv_heads=2), 0.3),     # k reaches the row width a quarter of the way down
    (dict(T=3000, k_top=6, n_q_heads=6, n_kv_heads=2, batch=2, local=True), 0.12),
])
def test_variable_k_follows_the_schedule(S, impl, kw, s):
    w = wl.generate(tc_spec(**kw))
    p = oracle_problem(w.spec)
    k_row = so.k_schedule(p, s)
    assert k_row.min() == 1 and k_row.max() == p.k_top and len(np.unique(k_row)) > 2
    # the library's own schedule is the same one
    sp = S.make_problem(*w.torch_tensors("cuda")[:2], block_q=64, block_k=64, k_top=p.k_top, causal=True)
    assert np.array_equal(S.k_schedule(sp, s).numpy(), k_row)
    variable_k_parity(S, w, k_row, impl=impl)


@pytest.mark.parametrize("impl", ["tensor", "generic"])
def test_variable_k_arbitrary_rows_and_clamping(S, impl):
    """k jumps up and down from one query block to the next (levels change with it) and holds
    entries outside 1 .. k_top, which are clamped."""
    w = wl.generate(tc_spec(T=6000, k_top=16, n_q_heads=8, n_kv_heads=2, anchors=True))
    nqb = -(-6000 // 64)
    rng = np.random.default_rng(3)
    k_row = rng.integers(1, 17, size=nqb).astype(np.int32)
    k_row[[5, 40]] = 0
    k_row[[6, 41]] = 99
    k_row[-1], k_row[-2] = 1, 16
    variable_k_parity(S, w, k_row, impl=impl)


def test_variable_k_non_causal_and_unequal_blocks_generic(S):
    w = wl.generate(small_spec(T=700, k_top=6))
    for causal, bq, bk in ((False, 32, 32), (True, 16, 32), (True, 1, 16)):
        p = oracle_problem(w.spec, block_q=bq, block_k=bk, causal=causal)
        nqb = so.num_query_blocks(p)
        k_row = (1 + np.arange(nqb) * 7 % 6).astype(np.int32)
        variable_k_parity(S, w, k_row, impl="generic", block_q=bq, block_k=bk, causal=causal, attention=bq > 1)


def test_variable_k_with_a_constant_schedule_is_the_fixed_k_build(S):
    w = wl.generate(tc_spec(T=4096, k_top=8))
    q, k, _ = w.torch_tensors("cuda")
    a = S.build_mask(q, k, block_q=64, block_k=64, k_top=8, want_scores=True)
    b = S.build_mask(q, k, block_q=64, block_k=64, k_top=8, want_scores=True,
                     k_row=torch.full((64,), 8, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert torch.equal(a.mask, b.mask) and torch.equal(a.scores, b.scores)
    assert a.stats().tiles_scored == b.stats().tiles_scored


@pytest.mark.parametrize("impl,kw,k_list", [
    ("generic", dict(T=2048, d=64, block=32, dtype="f32", n_q_heads=2, n_kv_heads=1, sink=False), [4, 2, 8]),
    ("generic", dict(T=5000, n_q_heads=3, n_kv_heads=1), [3, 6, 12]),
    ("tensor", dict(T=5000, n_q_heads=7, n_kv_heads=1), [3, 6, 12]),
    ("tensor", dict(T=8192, n_q_heads=4, n_kv_heads=2, anchors=True), [32, 16, 8, 1]),
])
def test_several_k_in_one_call(S, impl, kw, k_list):
    """Every slab of the several-k build against the oracle's mask for that k; the generic kernel
    scores a (row, block) tile once for all k, which the tile counter shows."""
    w = wl.generate(tc_spec(k_top=max(k_list), **kw))
    spec = w.spec
    q, k, _ = w.torch_tensors("cuda")
    res = S.build_masks(q, k, k_list, block_q=spec.block, block_k=spec.block, impl=impl, want_scores=True)
    torch.cuda.synchronize()
    st = res.stats()
    assert st.error == 0, f"device error {st.error} (info {st.error_info:#x})"
    p = oracle_problem(spec)
    ora = so.build_mask_rows_multi(p, w.q, w.k, k_list, want_scores=True)
    mask = res.mask.cpu().numpy().reshape(len(k_list), -1, p.k_top)
    sc = res.scores.cpu().numpy().reshape(mask.shape)
    all_same = True
    for i, ki in enumerate(k_list):
        report = compare_masks(mask[i], {"mask": ora["mask"][i], "min_gap": ora["min_gap"][i]})
        assert report["bad"] == 0, (ki, report)
        assert (mask[i][:, ki:] == -1).all()
        same = (mask[i] == ora["mask"][i]).all(axis=1)
        all_same &= bool(same.all()) and bool((ora["min_gap"][i] >= 1e-5).all())
        fin = np.isfinite(ora["scores"][i][same])
        np.testing.assert_allclose(sc[i][same][fin], ora["scores"][i][same][fin], rtol=2e-5, atol=2e-5)
        # the slab is what the single-k entry point gives
        one = S.build_mask(q, k, block_q=spec.block, block_k=spec.block, k_top=ki, impl=impl)
        assert torch.equal(one.mask, res.mask[i][..., :ki])
    assert st.rows == mask.shape[1] * (len(k_list) if impl == "tensor" else 1)
    if all_same:  # both kernels score a (row, block) tile once for all k: the oracle's union count
        separate = sum(int(so.build_mask_rows(oracle_problem(spec, k_top=ki), w.q, w.k)["tiles"].sum()) for ki in k_list)
        assert st.tiles_scored == int(ora["tiles"].sum()) < separate
        if impl == "tensor":  # with the small workspace only: one launch per k, nothing shared, same masks
            res2 = S.build_masks(q, k, k_list, block_q=spec.block, block_k=spec.block, impl=impl, share=False)
            torch.cuda.synchronize()
            assert torch.equal(res2.mask, res.mask) and res2.stats().tiles_scored == separate


def test_mask_tensor_core_repeats_bit_for_bit(S):
    """Many short groups per CTA with mixed group sizes (7 heads per kv head: groups of 4 and 3),
    k changing from one query block to the next and short lists: the case in which a warp with
    nothing to do in a list runs ahead of the others. Twenty launches must all give the oracle's
    rows (the kernel's roles meet only on barriers, so a lost ordering shows up as a rare wrong
    or missing row, not every time)."""
    w = wl.generate(tc_spec(T=2500, k_top=9, n_q_heads=14, n_kv_heads=2, batch=3, local=True))
    spec = w.spec
    p = oracle_problem(spec)
    nqb = so.num_query_blocks(p)
    k_row = (1 + (np.arange(nqb) * 5) % 9).astype(np.int32)
    ora = so.build_mask_rows_var(p, w.q, w.k, k_row)
    ok_rows = ora["min_gap"] >= 1e-5
    q, k, _ = w.torch_tensors("cuda")
    k_dev = torch.from_numpy(k_row).cuda()
    first = None
    for it in range(20):
        res = S.build_mask(q, k, block_q=64, block_k=64, k_top=9, impl="tensor", k_row=k_dev, want_scores=True)
        torch.cuda.synchronize()
        st = res.stats()
        assert st.error == 0, f"launch {it}: device error {st.error} (info {st.error_info:#x})"
        mask = res.mask.cpu().numpy().reshape(-1, 9)
        assert (mask[ok_rows] == ora["mask"][ok_rows]).all(), f"launch {it}"
        if first is None:
            first = (mask, res.scores.cpu().numpy())
        else:
            assert np.array_equal(mask, first[0]) and np.array_equal(res.scores.cpu().numpy(), first[1]), f"launch {it}"


def test_several_k_tensor_core_repeats_bit_for_bit(S):
    """The several-k launch (shared score memory, a group walked once per k) on many short groups
    of mixed size: ten launches, every slab the oracle's rows every time, and the same tile count."""
    w = wl.generate(tc_spec(T=2500, k_top=9, n_q_heads=14, n_kv_heads=2, batch=3, local=True))
    spec = w.spec
    ks = [3, 9, 5]
    ora = so.build_mask_rows_multi(oracle_problem(spec), w.q, w.k, ks)
    q, k, _ = w.torch_tensors("cuda")
    tiles = None
    for it in range(10):
        res = S.build_masks(q, k, ks, block_q=64, block_k=64, impl="tensor")
        torch.cuda.synchronize()
        st = res.stats()
        assert st.error == 0, f"launch {it}: device error {st.error} (info {st.error_info:#x})"
        mask = res.mask.cpu().numpy().reshape(len(ks), -1, 9)
        for i in range(len(ks)):
            ok_rows = ora["min_gap"][i] >= 1e-5
            assert (mask[i][ok_rows] == ora["mask"][i][ok_rows]).all(), f"launch {it}, k = {ks[i]}"
        tiles = st.tiles_scored if tiles is None else tiles
        assert st.tiles_scored == tiles


def test_a_bounded_wait_that_runs_out_is_reported(S):
    """The diagnostic kernel waits on a barrier nothing arrives at; after its limit the wait gives
    up the way every wait of the tensor-core kernels would: error word, abort flag, the warp
    leaves together, the kernel returns, and the host reads STREAM_ERR_DEVICE_CHECK. The context
    stays usable: a mask build right after it gives the oracle's rows."""
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    S.stream_selftest_bounded_wait(1_000_000, ws, ws.numel())   # about half a millisecond
    with pytest.raises(S.StreamError) as e:
        S.stream_read_stats(ws)
    assert e.value.status == S.STREAM_ERR_DEVICE_CHECK
    words = ws.cpu().numpy().view(np.uint64)
    assert words[0] == 1 and words[1] == 0          # abort flag raised; the wait did not succeed
    assert ws.cpu().numpy().view(np.uint32)[4] == 901
    w = wl.generate(tc_spec(T=2048, k_top=4))
    assert_mask_parity(S, w, None, impl="tensor", score_cache=False)


@pytest.mark.gpu
def test_unit_rate_probe_and_fetch_counter(S):
    """The measurement aid returns the two unit rates in the range this architecture can have
    (a tcgen05.mma of M = 128, N = 64, K = 16 needs at least its 32 tensor-core clocks; the TMA
    unit of one SM brings some tens of bytes per clock from L2), leaves the context usable, and the
    tensor-core block kernel's fetch counter lies between a quarter of the tiles scored (every
    fetched tile shared by the four heads of a kv head) and all of them."""
    r = S.probe_unit_rates()
    assert r.error == 0
    assert 32.0 <= r.mma_cycles_m128n64 <= 80.0, r.mma_cycles_m128n64
    assert 16.0 <= r.tma_bytes_per_clk <= 128.0, r.tma_bytes_per_clk
    w = wl.generate(tc_spec(T=4096, k_top=8, n_q_heads=8, n_kv_heads=2))
    q, k, _ = w.torch_tensors("cuda")
    res = S.build_mask(q, k, block_q=64, block_k=64, k_top=8, impl="tensor")
    st = res.stats()
    q_tiles = 8 * 64   # one query tile per row
    assert st.tiles_scored // 4 + q_tiles <= st.tiles_fetched <= st.tiles_scored + q_tiles, (st.tiles_fetched, st.tiles_scored)


def integer_workload(spec, lo=-2, hi=2):
    """Q and K with small integer entries (exact in bf16 and fp32): every dot product is an integer
    that fp32 accumulation and the oracle's fp64-then-round give alike, so tile maxima coincide
    exactly on both sides and many branches tie."""
    w = wl.generate(spec, with_v=False)
    rng = np.random.default_rng(spec.seed + 1000)
    def ints(shape):
        x = rng.integers(lo, hi + 1, size=shape).astype(np.float32)
        return wl.to_bf16_bits(x) if spec.dtype == "bf16" else x
    w.q = ints(w.q.shape)
    w.k = ints(w.k.shape)
    return w


@pytest.mark.gpu
@pytest.mark.parametrize("kw,impl,bq", [
    (dict(T=4096, k_top=8, n_q_heads=4, n_kv_heads=1), "tensor", 64),     # tcgen05 block kernel, 3 levels
    (dict(T=8192, k_top=32, n_q_heads=8, n_kv_heads=2), "tensor", 64),    # k = 32: all 64 candidates of a level compete
    (dict(T=5000, k_top=5, n_q_heads=3, n_kv_heads=1), "tensor", 64),     # ragged T, odd k
    (dict(T=4096, k_top=8, n_q_heads=4, n_kv_heads=1), "generic", 64),    # fp32-FMA kernel on the same inputs
    (dict(T=2048, k_top=16, n_q_heads=2, n_kv_heads=1), "auto", 1),       # per-token tensor-core kernel
])
def test_exact_ties_are_broken_by_block_index(S, kw, impl, bq):
    """With integer inputs the scores are exact on both sides and ties between branches are the
    rule, so nothing is exempt: every row must be the oracle's row, which keeps, among equal
    scores, the lower block index - and the scores of the kept blocks must be equal bit for bit."""
    spec = tc_spec(**kw)
    w = integer_workload(spec)
    res = run_mask(S, w, impl=impl, block_q=bq, want_scores=True)
    st = res.stats()
    assert st.error == 0
    mask = res.mask.cpu().numpy()
    flat = mask.reshape(-1, mask.shape[-1])
    p = oracle_problem(spec, block_q=bq)
    n_rows = flat.shape[0]
    rows = None if n_rows <= 4096 else np.unique(np.concatenate([np.arange(64), np.arange(n_rows - 64, n_rows),
                                                                  np.random.default_rng(3).choice(n_rows, 2048, replace=False)]))
    ora = so.build_mask_rows(p, w.q, w.k, rows, want_scores=True)
    got = flat if rows is None else flat[rows]
    assert (ora["min_gap"] < TIE_GAP).mean() > 0.1          # the case is what it says: exact ties at the cut are common
    np.testing.assert_array_equal(got, ora["mask"])
    sc = res.scores.cpu().numpy().reshape(-1, mask.shape[-1])
    sc = sc if rows is None else sc[rows]
    np.testing.assert_array_equal(sc, ora["scores"])


@pytest.mark.gpu
def test_exact_ties_in_the_several_k_and_variable_k_builds(S):
    """The same integer inputs through the several-k build (scores taken from the score memory in
    the later passes) and the variable-k build: every row, every k, bit for bit."""
    spec = tc_spec(T=4096, k_top=16, n_q_heads=8, n_kv_heads=2)
    w = integer_workload(spec)
    q, k, _ = w.torch_tensors("cuda")
    p = oracle_problem(spec)
    k_list = [16, 8, 3]
    res = S.build_masks(q, k, k_list, block_q=64, block_k=64, impl="tensor", want_scores=True)
    torch.cuda.synchronize()
    assert res.stats().error == 0
    ora = so.build_mask_rows_multi(p, w.q, w.k, k_list, want_scores=True)
    np.testing.assert_array_equal(res.mask.cpu().numpy().reshape(len(k_list), -1, p.k_top), ora["mask"])
    np.testing.assert_array_equal(res.scores.cpu().numpy().reshape(len(k_list), -1, p.k_top), ora["scores"])
    nqb = so.num_query_blocks(p)
    k_row = (1 + (np.arange(nqb) * 5) % 16).astype(np.int32)
    var = S.build_mask(q, k, block_q=64, block_k=64, k_top=16, k_row=torch.from_numpy(k_row).cuda(), impl="tensor", want_scores=True)
    torch.cuda.synchronize()
    assert var.stats().error == 0
    orv = so.build_mask_rows_var(p, w.q, w.k, k_row, want_scores=True)
    np.testing.assert_array_equal(var.mask.cpu().numpy().reshape(-1, p.k_top), orv["mask"])
    np.testing.assert_array_equal(var.scores.cpu().numpy().reshape(-1, p.k_top), orv["scores"])
