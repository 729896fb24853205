"""Pins for the CPU oracle: it is checked against things other than itself.

Hand-worked example, brute-force block scores, exact top-k for one level, invariants of
Algorithm 2, a differently structured simulation, and dense attention from a library routine.
"""
import math
import os
import zlib

import numpy as np
import pytest
import torch

from oracle import stream_oracle as so
from paper_2510_19875_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    return wl.to_bf16_bits(np.asarray(x, np.float32))


def bits_to_f32(a):
    return (a.astype(np.uint32) << 16).view(np.float32) if a.dtype == np.uint16 else a


def grid_inputs(rng, shape, dtype, step=1 / 16, span=3.0):
    """Random values on a coarse grid: every dot product is exact in fp32 and fp64."""
    x = np.clip(np.round(rng.standard_normal(shape) / step) * step, -span, span).astype(np.float32)
    return x if dtype == "f32" else bf16_bits(x)


# ---------------------------------------------------------------------------------------------
# An independent restatement of Algorithm 2, structured differently from the C oracle: nodes are
# explicit Python lists of block ids, scores come from one dense T_p x T_p product.
# ---------------------------------------------------------------------------------------------
def dense_scores(p, q, k, b, h):
    """(allowed[T_p, T_p], S[T_p, T_p] in fp32) for one head, padded with zeros."""
    l = math.lcm(p.block_q, p.block_k)
    Tp = -(-p.T // l) * l
    g = h // (p.n_q_heads // p.n_kv_heads)
    Q = np.zeros((Tp, p.d)), np.zeros((Tp, p.d))
    Qp, Kp = Q
    Qp[: p.T] = bits_to_f32(q[b, h]).astype(np.float64)
    Kp[: p.T] = bits_to_f32(k[b, g]).astype(np.float64)
    S = (Qp @ Kp.T).astype(np.float32)
    tq, tk = np.arange(Tp)[:, None], np.arange(Tp)[None, :]
    allowed = (tq < p.T) & (tk < p.T)
    if p.causal:
        allowed &= tk <= tq
    return allowed, S, Tp


def block_score_table(p, q, k, b, h):
    """Brute-force alpha(Q_i, K_j) under the mask (-inf where nothing is allowed), Eq. 4."""
    allowed, S, Tp = dense_scores(p, q, k, b, h)
    nq, nk = Tp // p.block_q, Tp // p.block_k
    Sm = np.where(allowed, S, -np.inf).reshape(nq, p.block_q, nk, p.block_k)
    return Sm.max(axis=(1, 3)), nq, nk


def simulate_row(p, table, nk, qb, n_it=None):
    """Returns (kept blocks, set of scored representatives, min relative gap)."""
    k = p.k_top
    valid = [np.isfinite(table[qb, r]) for r in range(nk)]
    nodes = [list(range((j * nk) // k, ((j + 1) * nk) // k)) for j in range(k)]
    if n_it is None:
        n_it = max(0, math.ceil(math.log2(nk))) if nk > 1 else 0
    scored, gap_min = set(), math.inf
    for _ in range(n_it):
        branches = []
        for node in nodes:
            half = (len(node) + 1) // 2
            branches += [node[:half], node[half:]]
        cand = []
        for hidx, br in enumerate(branches):
            reps = [r for r in br if valid[r]]
            if reps:
                scored.add(reps[0])
                cand.append((-float(table[qb, reps[0]]), hidx))
            else:
                cand.append((math.inf, hidx))
        cand.sort()
        a, c = -cand[k - 1][0], -cand[k][0]
        if math.isfinite(a) and math.isfinite(c):
            den = max(abs(np.float32(a)), abs(np.float32(c)))
            gap_min = min(gap_min, float((np.float32(a) - np.float32(c)) / den) if den > 0 else 0.0)
        nodes = [branches[hidx] for hidx in sorted(hidx for _, hidx in cand[:k])]
    kept = sorted(next(r for r in node if valid[r]) for node in nodes if any(valid[r] for r in node))
    return kept, scored, gap_min


def padded(row, k):
    return list(row) + [-1] * (k - len(row))


RANDOM_CASES = [
    # (B, H, G, T, d, bq, bk, k, causal, dtype)
    (1, 1, 1, 32, 2, 1, 1, 2, True, "f32"),
    (1, 1, 1, 64, 3, 4, 4, 4, True, "f32"),
    (1, 2, 1, 61, 3, 4, 4, 3, True, "bf16"),      # ragged T, odd k, GQA
    (2, 4, 2, 48, 4, 2, 2, 5, True, "f32"),       # batch + GQA + odd node sizes
    (1, 1, 1, 40, 2, 4, 2, 3, True, "f32"),       # b_q > b_k
    (1, 1, 1, 40, 2, 2, 4, 3, True, "bf16"),      # b_q < b_k
    (1, 1, 1, 37, 2, 3, 2, 4, True, "f32"),       # lcm padding
    (1, 2, 2, 64, 2, 4, 4, 4, False, "f32"),      # non-causal (HiP, Algorithm 1)
    (1, 1, 1, 24, 2, 2, 2, 16, True, "f32"),      # k > N_k
    (1, 1, 1, 56, 2, 1, 1, 7, True, "f32"),       # node sizes 8 with k = 7
    (1, 1, 1, 16, 1, 1, 1, 1, True, "f32"),       # k = 1
]


def case_seed(case) -> int:
    """The same seed in every process (Python randomises hash() of strings per run)."""
    return zlib.crc32(repr(case).encode())


@pytest.mark.parametrize("case", RANDOM_CASES)
def test_matches_independent_simulation(case):
    B, H, G, T, d, bq, bk, k, causal, dtype = case
    rng = np.random.default_rng(case_seed(case))
    for rep in range(3):
        step = 1.0 if rep == 0 else 1 / 16  # integer inputs give many exact ties
        q = grid_inputs(rng, (B, H, T, d), dtype, step)
        kk = grid_inputs(rng, (B, G, T, d), dtype, step)
        p = so.OracleProblem(B, H, G, T, d, bq, bk, k, causal, dtype)
        got = so.build_mask_rows(p, q, kk, want_scores=True)
        nq_rows = so.num_query_blocks(p)
        assert got["mask"].shape == (B * H * nq_rows, k)
        for b in range(B):
            for h in range(H):
                table, _, nk = block_score_table(p, q, kk, b, h)
                for qb in range(nq_rows):
                    kept, scored, gap = simulate_row(p, table, nk, qb)
                    i = (b * H + h) * nq_rows + qb
                    assert got["mask"][i].tolist() == padded(kept, k), (case, b, h, qb)
                    assert got["tiles"][i] == len(scored)
                    assert got["min_gap"][i] == pytest.approx(gap, rel=1e-6) or (math.isinf(gap) and math.isinf(got["min_gap"][i]))
                    assert got["scores"][i, : len(kept)].tolist() == [float(table[qb, r]) for r in kept]


def test_hand_example():
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "hand_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line in ("case", "case_var"):
            cur = {"rows": {}}
            cases.append(cur)
        elif line.startswith("k_row:"):
            cur["k_row"] = [int(x) for x in line[6:].split()]
        elif line.startswith("K:"):
            cur["K"] = [float(x) for x in line[2:].split()]
        else:
            qb, vals = line.split(":")
            cur["rows"][int(qb)] = [int(x) for x in vals.split()]
    assert len(cases) == 3 and sum("k_row" in c for c in cases) == 1
    for c in cases:
        K = np.array(c["K"], np.float32).reshape(1, 1, 8, 1)
        Q = np.ones((1, 1, 8, 1), np.float32)
        p = so.OracleProblem(1, 1, 1, 8, 1, 1, 1, 2, True, "f32")
        if "k_row" in c:
            mask = so.build_mask_rows_var(p, Q, K, np.array(c["k_row"], np.int32))["mask"]
        else:
            mask = so.build_mask_rows(p, Q, K)["mask"]
        for qb, want in c["rows"].items():
            assert mask[qb].tolist() == want


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("T,bq,bk", [(64, 8, 8), (61, 8, 8), (60, 4, 6), (30, 1, 4)])
def test_tile_score_is_masked_max_dot_product(dtype, causal, T, bq, bk):
    """Eq. 4 under the mask, by brute force; integer inputs make every sum exact."""
    rng = np.random.default_rng(7)
    q = grid_inputs(rng, (1, 2, T, 5), dtype, 1.0)
    k = grid_inputs(rng, (1, 1, T, 5), dtype, 1.0)
    p = so.OracleProblem(1, 2, 1, T, 5, bq, bk, 2, causal, dtype)
    for h in range(2):
        table, nq, nk = block_score_table(p, q, k, 0, h)
        for qb in range(so.num_query_blocks(p)):
            for r in range(nk):
                assert so.tile_score(p, q, k, 0, h, qb, r) == table[qb, r]


def test_tile_score_fp64_accumulation_rounds_once():
    """A sum that fp32 accumulation gets wrong: 2^24 + 1 - 2^24 ... the oracle must return 1."""
    q = np.array([[[[1.0, 1.0, 1.0]]]], np.float32)
    k = np.array([[[[16777216.0, 1.0, -16777216.0]]]], np.float32)
    p = so.OracleProblem(1, 1, 1, 1, 3, 1, 1, 1, True, "f32")
    assert so.tile_score(p, q, k, 0, 0, 0, 0) == 1.0


@pytest.mark.parametrize("causal", [True, False])
def test_single_level_is_exact_topk(causal):
    """N_k = 2k: one split reaches single blocks, so the row is the exact top-k of block scores."""
    rng = np.random.default_rng(11)
    T, b, k, d = 128, 4, 16, 6
    q = grid_inputs(rng, (1, 1, T, d), "f32", 1 / 8)
    kk = grid_inputs(rng, (1, 1, T, d), "f32", 1 / 8)
    p = so.OracleProblem(1, 1, 1, T, d, b, b, k, causal, "f32")
    mask = so.build_mask_rows(p, q, kk)["mask"]
    table, nq, nk = block_score_table(p, q, kk, 0, 0)
    assert nk == 2 * k
    for qb in range(nq):
        valid = [r for r in range(nk) if np.isfinite(table[qb, r])]
        best = sorted(valid, key=lambda r: (-table[qb, r], r))[:k]
        assert mask[qb].tolist() == padded(sorted(best), k)


def test_k_equal_one_is_binary_descent():
    rng = np.random.default_rng(5)
    T = 64
    K = rng.permutation(T).astype(np.float32).reshape(1, 1, T, 1)  # distinct scores
    Q = np.ones((1, 1, T, 1), np.float32)
    p = so.OracleProblem(1, 1, 1, T, 1, 1, 1, 1, True, "f32")
    mask = so.build_mask_rows(p, Q, K)["mask"]
    for qb in range(T):
        lo, hi = 0, T - 1
        while lo < hi:  # compare the first block of each half; right half only if it is causal
            mid = (lo + hi) // 2
            if mid + 1 <= qb and K[0, 0, mid + 1, 0] > K[0, 0, lo, 0]:
                lo = mid + 1
            else:
                hi = mid
        assert mask[qb, 0] == lo


@pytest.mark.parametrize("spec_kw", [
    dict(T=1024, d=16, block=16, k_top=8, n_q_heads=4, n_kv_heads=2, dtype="bf16", sink=True, local=True),
    dict(T=1000, d=8, block=8, k_top=5, n_q_heads=2, n_kv_heads=1, dtype="f32", anchors=True, sink=True),
    dict(T=512, d=8, block=8, k_top=4, n_q_heads=2, n_kv_heads=2, batch=2, dtype="bf16", needle=True),
])
def test_invariants_on_structured_inputs(spec_kw):
    spec = wl.WorkloadSpec(name="t", seed=9, batch=spec_kw.pop("batch", 1), **{
        "n_q_heads": 1, "n_kv_heads": 1, "T": 64, "d": 4, "block": 4, "k_top": 2, "dtype": "f32", **spec_kw})
    w = wl.generate(spec, with_v=False)
    p = so.OracleProblem(spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d, spec.block, spec.block,
                         spec.k_top, True, spec.dtype)
    res = so.build_mask_rows(p, w.q, w.k)
    nqb = so.num_query_blocks(p)
    for i, row in enumerate(res["mask"]):
        qb = i % nqb
        kept = row[row >= 0]
        assert (row[len(kept):] == -1).all()                       # padding only at the end
        assert (np.diff(kept) > 0).all()                           # strictly ascending, no repeats
        last_tok = min(qb * spec.block + spec.block - 1, spec.T - 1)
        assert (kept * spec.block <= last_tok).all()               # causal: no block after the query
        n_valid = last_tok // spec.block + 1
        assert len(kept) == min(spec.k_top, n_valid)               # exactly min(k, causal blocks)
    # extra iterations, fewer (but enough) iterations and the score cache change nothing
    L = math.ceil(math.log2(max(1, -(-nqb // spec.k_top)))) if nqb > spec.k_top else 0
    for kw in (dict(n_it=L), dict(n_it=L + 7), dict(score_cache=True)):
        assert (so.build_mask_rows(p, w.q, w.k, **kw)["mask"] == res["mask"]).all()
    # scaling Q by two is exact in floating point and cannot change any ordering
    q2 = (bits_to_f32(w.q) * 2).astype(np.float32)
    q2 = q2 if spec.dtype == "f32" else bf16_bits(q2)
    assert (so.build_mask_rows(p, q2, w.k)["mask"] == res["mask"]).all()


def test_unscored_key_blocks_do_not_matter():
    rng = np.random.default_rng(21)
    T, b, k, d = 256, 4, 4, 3
    q = grid_inputs(rng, (1, 1, T, d), "f32", 1 / 16)
    kk = grid_inputs(rng, (1, 1, T, d), "f32", 1 / 16)
    p = so.OracleProblem(1, 1, 1, T, d, b, b, k, True, "f32")
    table, nq, nk = block_score_table(p, q, kk, 0, 0)
    qb = nq - 1
    kept, scored, _ = simulate_row(p, table, nk, qb)
    assert len(scored) < nk // 2  # the hierarchy looks at a small part of the keys
    k2 = kk.copy()
    for r in range(nk):
        if r not in scored:
            k2[0, 0, r * b:(r + 1) * b] = 100.0 * rng.standard_normal((b, d)).astype(np.float32)
    rows = np.array([qb])
    assert (so.build_mask_rows(p, q, k2, rows)["mask"] == so.build_mask_rows(p, q, kk, rows)["mask"]).all()


def test_row_subset_and_gqa_head_mapping():
    rng = np.random.default_rng(3)
    H, G, T, d, b, k = 4, 2, 64, 4, 4, 3
    q = grid_inputs(rng, (1, H, T, d), "f32")
    kk = grid_inputs(rng, (1, G, T, d), "f32")
    p = so.OracleProblem(1, H, G, T, d, b, b, k, True, "f32")
    full = so.build_mask_rows(p, q, kk)["mask"]
    rows = np.array([5, 63, 17, 40])
    assert (so.build_mask_rows(p, q, kk, rows)["mask"] == full[rows]).all()
    # query head h must read kv head h // (H / G): compare with single-head problems
    p1 = so.OracleProblem(1, 1, 1, T, d, b, b, k, True, "f32")
    nqb = T // b
    for h in range(H):
        solo = so.build_mask_rows(p1, np.ascontiguousarray(q[:, h:h + 1]), np.ascontiguousarray(kk[:, h // 2:h // 2 + 1]))["mask"]
        assert (solo == full[h * nqb:(h + 1) * nqb]).all()


# ---------------------------------------------------------------------------------------------
# Sparse attention (Eq. 2)
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("causal", [True, False])
def test_full_mask_equals_dense_attention(dtype, causal):
    """k >= N_k keeps every allowed block, so Eq. 2 must reduce to Eq. 1 (library SDPA, fp64)."""
    rng = np.random.default_rng(13)
    B, H, G, T, d, b = 2, 4, 2, 96, 8, 8
    q = grid_inputs(rng, (B, H, T, d), dtype, 1 / 16)
    kk = grid_inputs(rng, (B, G, T, d), dtype, 1 / 16)
    v = grid_inputs(rng, (B, G, T, d), dtype, 1 / 16)
    p = so.OracleProblem(B, H, G, T, d, b, b, T // b + 3, causal, dtype)
    mask = so.build_mask_rows(p, q, kk)["mask"]
    nqb = T // b
    for i, row in enumerate(mask):
        n_valid = (i % nqb) + 1 if causal else nqb
        assert row.tolist() == padded(range(n_valid), p.k_top)
    out = so.sparse_attention_rows(p, q, kk, v, mask).reshape(B, H, T, d)
    tq = torch.from_numpy(bits_to_f32(q).astype(np.float64))
    tk = torch.from_numpy(bits_to_f32(kk).astype(np.float64)).repeat_interleave(H // G, dim=1)
    tv = torch.from_numpy(bits_to_f32(v).astype(np.float64)).repeat_interleave(H // G, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=causal).numpy()
    np.testing.assert_allclose(out, ref, rtol=1e-10, atol=1e-12)


def test_sparse_attention_matches_direct_sum_and_handles_empty_tokens():
    rng = np.random.default_rng(17)
    T, d, bq, bk, k = 30, 3, 4, 6, 2  # b_q != b_k: early tokens of a query block may see no key
    q = grid_inputs(rng, (1, 1, T, d), "f32")
    kk = grid_inputs(rng, (1, 1, T, d), "f32")
    v = grid_inputs(rng, (1, 1, T, d), "f32")
    p = so.OracleProblem(1, 1, 1, T, d, bq, bk, k, True, "f32")
    nqb = so.num_query_blocks(p)
    mask = np.full((nqb, k), -1, np.int32)
    for qb in range(nqb):
        mask[qb, 0] = (qb * bq + bq - 1) // bk if (qb * bq + bq - 1) < T else (T - 1) // bk
    mask[0, 0] = 0
    mask[2, :] = [1, -1]  # block 1 = tokens 6..11, query block 2 = tokens 8..11: all see something
    mask[1, :] = [1, -1]  # query block 1 = tokens 4..7: tokens 4, 5 see no key of block 1
    scale = 0.37
    out = so.sparse_attention_rows(p, q, kk, v, mask, scale=scale)
    for qb in range(nqb):
        for m in range(bq):
            t = qb * bq + m
            keys = [r * bk + n for r in mask[qb] if r >= 0 for n in range(bk) if r * bk + n < T and r * bk + n <= t]
            if t >= T or not keys:
                assert (out[qb, m] == 0).all()
                continue
            logit = scale * (kk[0, 0, keys].astype(np.float64) @ q[0, 0, t].astype(np.float64))
            w = np.exp(logit - logit.max())
            w /= w.sum()
            np.testing.assert_allclose(out[qb, m], w @ v[0, 0, keys].astype(np.float64), rtol=1e-12, atol=1e-14)
    assert (out[1, 0] == 0).all() and (out[1, 1] == 0).all() and out[1, 2].any()


def test_default_scale_is_inverse_sqrt_d():
    rng = np.random.default_rng(19)
    q = grid_inputs(rng, (1, 1, 16, 4), "f32")
    kk = grid_inputs(rng, (1, 1, 16, 4), "f32")
    v = grid_inputs(rng, (1, 1, 16, 4), "f32")
    p = so.OracleProblem(1, 1, 1, 16, 4, 4, 4, 2, True, "f32")
    mask = so.build_mask_rows(p, q, kk)["mask"]
    a = so.sparse_attention_rows(p, q, kk, v, mask)
    b = so.sparse_attention_rows(p, q, kk, v, mask, scale=0.5)
    assert (a == b).all()


def test_vertical_scores_are_column_sums_with_library_kurtosis():
    """Pins for the vertical scores: numpy's bincount for the sums, scipy's Pearson kurtosis for
    the fourth-moment ratio, and a hand-worked row."""
    from scipy import stats

    p = so.OracleProblem(2, 2, 1, 96, 4, 8, 8, 3, True, "f32")
    nq = nk = 12
    rng = np.random.default_rng(3)
    mask = rng.integers(-1, nk, size=(2 * 2 * nq, 3)).astype(np.int32)
    scores = rng.standard_normal(mask.shape).astype(np.float32)
    vert, kurt = so.vertical_scores(p, mask)
    wvert, wkurt = so.vertical_scores(p, mask, scores)
    for h in range(4):
        rows = mask[h * nq:(h + 1) * nq]
        keep = rows >= 0
        np.testing.assert_array_equal(vert[h], np.bincount(rows[keep], minlength=nk))
        np.testing.assert_allclose(wvert[h], np.bincount(rows[keep], weights=scores[h * nq:(h + 1) * nq][keep].astype(np.float64), minlength=nk), rtol=1e-12, atol=1e-12)
        assert kurt[h] == pytest.approx(stats.kurtosis(vert[h], fisher=False, bias=True), rel=1e-12)
        assert wkurt[h] == pytest.approx(stats.kurtosis(wvert[h], fisher=False, bias=True), rel=1e-12)
    # by hand: one head, 4 key blocks, every query block keeps block 0 and itself -> v = [4, 1, 1, 1]
    p1 = so.OracleProblem(1, 1, 1, 32, 4, 8, 8, 2, True, "f32")
    m1 = np.array([[0, -1], [0, 1], [0, 2], [0, 3]], np.int32)
    v1, k1 = so.vertical_scores(p1, m1)
    assert v1.tolist() == [[4.0, 1.0, 1.0, 1.0]]
    # mean 1.75, deviations (2.25, -.75, -.75, -.75): m2 = 1.6875, m4 = 6.64453125 -> 2.3333...
    assert k1[0] == pytest.approx(6.64453125 / 1.6875 ** 2, rel=1e-14)
    assert so.vertical_scores(p1, np.array([[0, -1], [1, -1], [2, -1], [3, -1]], np.int32))[1][0] == 0.0  # flat


def test_mask_difference_is_the_row_wise_set_difference():
    """Pins: numpy's setdiff1d per row (the rows hold distinct blocks), order and scores carried
    from the first mask, and a hand-worked row."""
    rng = np.random.default_rng(9)
    n, ka, kb, nk = 40, 6, 3, 20
    a = np.stack([rng.permutation(nk)[:ka] for _ in range(n)]).astype(np.int32)
    b = np.stack([rng.permutation(nk)[:kb] for _ in range(n)]).astype(np.int32)
    a[rng.random(a.shape) < 0.2] = -1
    b[rng.random(b.shape) < 0.2] = -1
    sc = rng.standard_normal(a.shape).astype(np.float32)
    diff, dsc = so.mask_difference(a, b, sc)
    for i in range(n):
        kept = diff[i][diff[i] >= 0]
        assert sorted(kept.tolist()) == np.setdiff1d(a[i][a[i] >= 0], b[i]).tolist()
        want = [x for x in a[i].tolist() if x >= 0 and x not in b[i].tolist()]      # order of the first mask
        assert kept.tolist() == want
        assert (diff[i][len(kept):] == -1).all() and (dsc[i][len(kept):] == -np.inf).all()
        assert dsc[i][: len(kept)].tolist() == [float(sc[i][a[i].tolist().index(x)]) for x in want]
    d, _ = so.mask_difference(np.array([[0, 3, 5, 9, -1, -1]], np.int32), np.array([[0, 9, -1]], np.int32))
    assert d.tolist() == [[3, 5, -1, -1, -1, -1]]


@pytest.mark.parametrize("case", RANDOM_CASES[:8])
def test_variable_k_rows_match_independent_simulation(case):
    """Each row of the variable-k build is Algorithm 2 with that row's own k: checked against the
    list-based simulation above, run with the row's k, on k_row values that include 1, k_top and
    out-of-range entries (clamped)."""
    import dataclasses

    B, H, G, T, d, bq, bk, k, causal, dtype = case
    rng = np.random.default_rng(case_seed(case) + 1)
    q = grid_inputs(rng, (B, H, T, d), dtype, 1 / 16)
    kk = grid_inputs(rng, (B, G, T, d), dtype, 1 / 16)
    p = so.OracleProblem(B, H, G, T, d, bq, bk, k, causal, dtype)
    nq_rows = so.num_query_blocks(p)
    k_row = rng.integers(1, k + 1, size=nq_rows).astype(np.int32)
    k_row[0], k_row[-1] = 0, k + 3  # clamped to 1 and k
    if nq_rows > 3:
        k_row[1], k_row[2] = 1, k
    got = so.build_mask_rows_var(p, q, kk, k_row, want_scores=True)
    assert got["mask"].shape == (B * H * nq_rows, k)
    for b in range(B):
        for h in range(H):
            table, _, nk = block_score_table(p, q, kk, b, h)
            for qb in range(nq_rows):
                kq = int(min(max(k_row[qb], 1), k))
                kept, scored, _ = simulate_row(dataclasses.replace(p, k_top=kq), table, nk, qb)
                i = (b * H + h) * nq_rows + qb
                assert got["mask"][i].tolist() == padded(kept, k), (case, b, h, qb, kq)
                assert got["tiles"][i] == len(scored)
                assert got["scores"][i, : len(kept)].tolist() == [float(table[qb, r]) for r in kept]
                assert np.isneginf(got["scores"][i, len(kept):]).all()


def test_variable_k_with_constant_schedule_is_the_fixed_k_build():
    rng = np.random.default_rng(11)
    p = so.OracleProblem(1, 2, 1, 96, 4, 4, 4, 3, True, "f32")
    q = grid_inputs(rng, (1, 2, 96, 4), "f32")
    k = grid_inputs(rng, (1, 1, 96, 4), "f32")
    a = so.build_mask_rows(p, q, k, want_scores=True)
    b = so.build_mask_rows_var(p, q, k, np.full(so.num_query_blocks(p), 3, np.int32), want_scores=True)
    for key in ("mask", "scores", "min_gap", "tiles"):
        np.testing.assert_array_equal(a[key], b[key])


@pytest.mark.parametrize("causal", [True, False])
def test_k_schedule_closed_form(causal):
    """k(q) = floor(1 + (n(q) - 1) s) with n(q) the row's allowed key blocks: q + 1 under a causal
    mask with equal blocks, all of them without one; clamped to k_top."""
    T, blk, k_top, s = 64 * 4 - 3, 4, 12, 0.25
    p = so.OracleProblem(1, 1, 1, T, 2, blk, blk, k_top, causal, "f32")
    got = so.k_schedule(p, s)
    nq = -(-T // blk)
    n = np.arange(1, nq + 1) if causal else np.full(nq, nq)
    want = np.clip(np.floor(1 + (n - 1) * s), 1, k_top).astype(np.int32)
    assert got.tolist() == want.tolist()
    assert got.max() == k_top and (not causal or got[0] == 1)  # the clamp is reached
    with pytest.raises(RuntimeError):
        so.k_schedule(p, 1.0)


@pytest.mark.parametrize("case", [RANDOM_CASES[1], RANDOM_CASES[3], RANDOM_CASES[6], RANDOM_CASES[7]])
def test_several_k_at_once_match_the_simulation_and_count_shared_tiles(case):
    """Mask i of the multi-k build is Algorithm 2 with k_list[i]; the tile count of a row is the
    size of the UNION of the representatives the simulation scores for the different k."""
    import dataclasses

    B, H, G, T, d, bq, bk, k, causal, dtype = case
    rng = np.random.default_rng(case_seed(case) + 2)
    q = grid_inputs(rng, (B, H, T, d), dtype, 1 / 16)
    kk = grid_inputs(rng, (B, G, T, d), dtype, 1 / 16)
    k_list = sorted({1, max(1, k // 2), k})
    p = so.OracleProblem(B, H, G, T, d, bq, bk, k, causal, dtype)
    got = so.build_mask_rows_multi(p, q, kk, k_list, want_scores=True)
    nq_rows = so.num_query_blocks(p)
    assert got["mask"].shape == (len(k_list), B * H * nq_rows, k)
    shared_less = False
    for b in range(B):
        for h in range(H):
            table, _, nk = block_score_table(p, q, kk, b, h)
            for qb in range(nq_rows):
                i = (b * H + h) * nq_rows + qb
                union, total = set(), 0
                for j, kj in enumerate(k_list):
                    kept, scored, _ = simulate_row(dataclasses.replace(p, k_top=kj), table, nk, qb)
                    assert got["mask"][j, i].tolist() == padded(kept, k), (case, b, h, qb, kj)
                    assert got["scores"][j, i, : len(kept)].tolist() == [float(table[qb, r]) for r in kept]
                    union |= scored
                    total += len(scored)
                assert got["tiles"][i] == len(union)
                shared_less |= len(union) < total
    assert shared_less  # the k do share representatives
    single = so.build_mask_rows(dataclasses.replace(p, k_top=k_list[-1]), q, kk)["mask"]
    np.testing.assert_array_equal(got["mask"][-1][:, : k_list[-1]], single)


@pytest.mark.parametrize("T,blk,s", [(8192, 32, 0.1), (1000, 32, 0.2), (131072, 64, 1 / 128), (4096, 64, 0.5)])
def test_k_schedule_ends_at_the_papers_formula(T, blk, s):
    """For the last query block of a causal pattern the row's own count of allowed blocks is
    ceil(T / b), so the schedule's last entry is the printed k = floor(1 + (T / b_q - 1) s)
    evaluated with that count (the two agree exactly when b divides T)."""
    n = -(-T // blk)
    p = so.OracleProblem(1, 1, 1, T, 2, blk, blk, n, True, "f32")  # k_top = n: no clamp from above
    got = so.k_schedule(p, s)
    assert got[-1] == int(math.floor(1 + (n - 1) * s))
    assert (np.diff(got) >= 0).all() and got[0] == 1  # grows down the pattern, one block at the top
    if T % blk == 0:
        assert got[-1] == max(1, min(int(1 + (T / blk - 1) * s), T // blk))


def test_effective_k_is_the_printed_formula():
    """Pins so.effective_k to values worked out by hand from k = floor(1 + (T / b_q - 1) s)
    (Section 4.2) and to the ends of k's range 1 .. floor(T / b_q) (Section 3)."""
    assert so.effective_k(1000, 32, 0.0) == 1             # s = 0: the smallest k
    assert so.effective_k(1024, 32, 1.0) == 32            # s = 1: every block, T / b_q
    assert so.effective_k(1000, 32, 1.0) == 31            # 1 + 30.25 = 31.25 -> 31 = floor(T / b_q)
    assert so.effective_k(8192, 32, 0.1) == 26            # 1 + 255 * 0.1 = 26.5
    assert so.effective_k(8192, 32, 0.5) == 128           # 1 + 127.5
    assert so.effective_k(20000, 32, 0.04) == 25          # 1 + 624 * 0.04 = 25.96
    assert so.effective_k(64, 64, 0.5) == 1               # one block
    assert so.effective_k(10, 64, 0.7) == 1               # less than one block: never below 1
    ks = [so.effective_k(10000, 32, s / 50) for s in range(51)]
    assert ks == sorted(ks) and ks[0] == 1 and ks[-1] == 312   # as printed, k grows with s
    for bad in (-0.1, 1.5, float("nan")):
        with pytest.raises(ValueError):
            so.effective_k(1000, 32, bad)
