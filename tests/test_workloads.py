"""The seeded input generators: deterministic, shaped as stated, and carrying the planted structure."""
import numpy as np
import pytest

from paper_2510_19875_b200 import workloads as wl


def f32(a):
    return (a.astype(np.uint32) << 16).view(np.float32) if a.dtype == np.uint16 else a


def small(name, **kw):
    return wl.SPECS[name].scaled(**kw)


def test_same_seed_same_bytes_and_heads_are_independent_streams():
    spec = small("gqa_layer_16k", T=512, n_q_heads=4, n_kv_heads=2)
    a, b = wl.generate(spec), wl.generate(spec)
    assert a.q.tobytes() == b.q.tobytes() and a.k.tobytes() == b.k.tobytes() and a.v.tobytes() == b.v.tobytes()
    c = wl.generate(spec.scaled(seed=spec.seed + 1))
    assert a.q.tobytes() != c.q.tobytes()
    assert a.q.shape == (1, 4, 512, 128) and a.k.shape == a.v.shape == (1, 2, 512, 128) and a.q.dtype == np.uint16


def test_config_shapes_match_the_five_workloads():
    s = wl.SPECS
    assert (s["single_head_fp32"].T, s["single_head_fp32"].d, s["single_head_fp32"].block, s["single_head_fp32"].k_top) == (2048, 64, 32, 8)
    assert (s["cot_layer_128k"].n_q_heads, s["cot_layer_128k"].n_kv_heads, s["cot_layer_128k"].T, s["cot_layer_128k"].k_top) == (32, 8, 131072, 32)
    assert (s["needle_stack_32k"].batch, s["needle_stack_32k"].n_q_heads, s["needle_stack_32k"].n_kv_heads) == (28, 28, 4)
    assert wl.SWEEP_T[-1] == 1 << 20 and s["sweep"].k_top == 32


def test_sink_key_and_query_shift():
    spec = small("sweep", T=256, n_q_heads=2, n_kv_heads=1)
    w = wl.generate(spec)
    k, q = f32(w.k)[0, 0], f32(w.q)[0]
    assert np.linalg.norm(k[0]) == pytest.approx(4 * 128 ** 0.5, rel=1e-2)
    u = k[0] / np.linalg.norm(k[0])
    assert (q @ u).mean() == pytest.approx(2.0, abs=0.2)      # every query leans on the sink direction
    assert abs((k[1:] @ u).mean()) < 0.3


def test_needle_block_and_last_queries_are_aligned():
    spec = small("needle_stack_32k", batch=1, T=2048, n_q_heads=2, n_kv_heads=1)
    w = wl.generate(spec)
    blk = w.notes[("needle_block", 0, 0)]
    assert 1 <= blk < spec.n_blocks // 2
    keys = f32(w.k)[0, 0, blk * 64:(blk + 1) * 64]
    n = keys[0] / np.linalg.norm(keys[0])
    cos_k = (keys @ n) / np.linalg.norm(keys, axis=1)
    assert cos_k.min() > 0.995
    qs = f32(w.q)[0, :, -128:]
    cos_q = (qs @ n) / np.linalg.norm(qs, axis=-1)
    assert np.allclose(cos_q, 0.9, atol=0.01)


def test_anchor_queries_reach_cosine_point_eight():
    spec = small("cot_layer_128k", T=4096, n_q_heads=1, n_kv_heads=1)
    w = wl.generate(spec)
    pos = w.notes[("anchors", 0, 0)]
    assert len(pos) == 64 and pos.min() >= 1 and len(set(pos.tolist())) == 64
    k, q = f32(w.k)[0, 0], f32(w.q)[0, 0]
    kn = k[pos] / np.linalg.norm(k[pos], axis=1, keepdims=True)
    cos = (q / np.linalg.norm(q, axis=1, keepdims=True)) @ kn.T          # [T, 64]
    causal = pos[None, :] < np.arange(spec.T)[:, None]
    best = np.where(causal, cos, -1).max(1)
    frac = (np.abs(best - 0.8) < 0.01).mean()
    assert 0.06 < frac < 0.14                                           # about 10 % of the queries


def test_bf16_cast_is_round_to_nearest_even():
    # 1 + 2^-8 and 1 + 3 * 2^-8 lie half-way between two bf16 values: ties go to the even mantissa
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, np.nextafter(np.float32(1.00390625), np.float32(2))], np.float32)
    assert f32(wl.to_bf16_bits(x)).tolist() == [1.0, 1.0, 1.015625, -2.5, 1.0078125]
