"""Shared by the test files: oracle problem from a workload spec, row sampling, mask comparison."""
import numpy as np

from oracle import stream_oracle as so

TIE_GAP = 1e-5  # rows whose k-th / (k+1)-th oracle score gap is below this (relative) are exempt


def oracle_problem(spec, *, block_q=None, block_k=None, k_top=None, causal=True):
    return so.OracleProblem(spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d, block_q or spec.block,
                            block_k or spec.block, k_top or spec.k_top, causal, spec.dtype)


def sample_rows(spec, n, seed=0):
    """Seeded sample of flat row ids that always holds the first and last 8 query blocks of head 0
    and of the last head."""
    nqb = spec.n_blocks
    total = spec.n_rows
    if n >= total:
        return np.arange(total, dtype=np.int64)
    rng = np.random.default_rng(seed)
    edge = [h * nqb + qb for h in (0, spec.batch * spec.n_q_heads - 1)
            for qb in list(range(min(8, nqb))) + list(range(max(0, nqb - 8), nqb))]
    rest = rng.choice(total, size=n, replace=False)
    return np.unique(np.concatenate([np.array(edge, np.int64), rest]))[: max(n, len(edge))]


def compare_masks(gpu_rows: np.ndarray, oracle: dict):
    """Bit-exact comparison row by row. Returns a dict of counts; ``bad`` must be 0."""
    same = (gpu_rows == oracle["mask"]).all(axis=1)
    exempt = oracle["min_gap"] < TIE_GAP
    return {
        "rows": int(same.shape[0]),
        "exempt": int(exempt.sum()),
        "exempt_and_different": int((~same & exempt).sum()),
        "bad": int((~same & ~exempt).sum()),
        "first_bad": int(np.nonzero(~same & ~exempt)[0][0]) if (~same & ~exempt).any() else -1,
    }


def check_mask_invariants(mask: np.ndarray, spec, *, block_q=None, block_k=None, causal=True):
    """Properties every row must have at any size: padding at the end, strictly ascending,
    causal, and exactly min(k, allowed blocks) entries. mask is [B, H, n_qb, k]."""
    bq, bk = block_q or spec.block, block_k or spec.block
    B, H, nqb, k = mask.shape
    kept = mask >= 0
    cnt = kept.sum(-1)
    # padding only at the end
    assert (kept[..., 1:] <= kept[..., :-1]).all()
    # strictly ascending among kept
    d = np.diff(mask.astype(np.int64), axis=-1)
    assert (d[kept[..., 1:]] > 0).all()
    qb = np.arange(nqb)
    last_tok = np.minimum(qb * bq + bq - 1, spec.T - 1) if causal else np.full(nqb, spec.T - 1)
    n_valid = last_tok // bk + 1
    assert (cnt == np.minimum(k, n_valid)[None, None, :]).all()
    top = np.where(kept, mask, -1).max(-1)
    assert (top <= (last_tok // bk)[None, None, :]).all()
