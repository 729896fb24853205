"""Host-side checks that need no GPU: the library loads, exports what the header declares, and
rejects bad arguments before anything is launched."""
import ctypes
import os
import re

import pytest

from paper_2510_19875_b200 import build as stream_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def S():
    stream_build.build_library()
    from paper_2510_19875_b200 import stream

    return stream


def declared_functions():
    names = []
    inc = os.path.join(ROOT, "include")
    for fn in sorted(os.listdir(inc)):
        text = open(os.path.join(inc, fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names += re.findall(r"\b(stream_[a-z_0-9]+)\s*\(", text)
    return sorted(set(names))


def test_library_exports_every_declared_symbol(S):
    lib = ctypes.CDLL(S.library_path())
    names = declared_functions()
    assert {"stream_build_mask", "stream_sparse_attention", "stream_workspace_bytes", "stream_run_host",
            "stream_host_staging_bytes", "stream_read_stats", "stream_last_error", "stream_version"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
        assert hasattr(S, n), f"binding lacks {n}"
    assert S.stream_version() >= 100


def good_problem(S, **kw):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=2, T=256, d=128, block_q=64, block_k=64, k_top=4, causal=1,
                dtype=S.STREAM_BF16, impl=0, q_stride_b=4 * 256 * 128, q_stride_h=256 * 128, q_stride_t=128,
                kv_stride_b=2 * 256 * 128, kv_stride_h=256 * 128, kv_stride_t=128)
    base.update(kw)
    return S.StreamProblem(**base)


@pytest.mark.parametrize("kw", [
    dict(batch=0), dict(n_kv_heads=3), dict(T=0), dict(d=0), dict(block_q=0), dict(block_k=-1), dict(k_top=0),
    dict(dtype=7), dict(impl=9), dict(causal=2), dict(q_stride_t=64), dict(kv_stride_h=-1),
])
def test_invalid_problem_is_rejected_on_the_host(S, kw):
    p = good_problem(S, **kw)
    assert S.stream_workspace_bytes(p) == 0
    assert S.stream_host_staging_bytes(p) == 0
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask(p, 256, 256, 256, None, 256, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
    assert S.stream_last_error() != ""


def test_null_pointers_and_workspace_are_checked_before_launch(S):
    p = good_problem(S)
    assert S.stream_workspace_bytes(p) >= 256
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask(p, None, 256, 256, None, 256, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
    for ws, nbytes in ((None, 256), (256, 8), (264, 4096)):  # missing, too small, misaligned
        with pytest.raises(S.StreamError) as e:
            S.stream_build_mask(p, 256, 256, 256, None, ws, nbytes, stream=0)
        assert e.value.status == S.STREAM_ERR_WORKSPACE
    with pytest.raises(S.StreamError) as e:
        S.stream_sparse_attention(p, 256, 256, None, 256, 0.0, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
    with pytest.raises(S.StreamError) as e:
        S.stream_run_host(p, 256, 256, 256, 256, 256, 0.0, None, 0, stream=0)
    assert e.value.status == S.STREAM_ERR_WORKSPACE


def test_unsupported_shapes_say_so(S):
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask(good_problem(S, k_top=5000), 256, 256, 256, None, 256, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_UNSUPPORTED
    # the tensor-core kernels take one shape only; asking for them elsewhere is an error, not a fallback
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask(good_problem(S, dtype=S.STREAM_F32, impl=2), 256, 256, 256, None, 256, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_UNSUPPORTED


def test_cpu_tensors_are_refused(S):
    import torch

    q = torch.zeros(1, 1, 64, 64)
    with pytest.raises(ValueError):
        S.build_mask(q, q, block_q=32, block_k=32, k_top=2)
    with pytest.raises(ValueError):
        S.sparse_attention(q, q, q, torch.zeros(1, 1, 2, 2, dtype=torch.int32), block_q=32, block_k=32)


def test_run_host_var_needs_a_schedule(S):
    p = good_problem(S)
    with pytest.raises(S.StreamError) as e:
        S.stream_run_host_var(p, 256, 256, 256, None, 256, 256, 0.0, 256, 1 << 30, stream=0)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG


def test_staging_size_covers_all_buffers(S):
    p = good_problem(S)
    e = 2
    need = (4 * 256 * 128 * e) * 2 + (2 * 256 * 128 * e) * 2 + 4 * 4 * 4 * 4 + 256
    assert S.stream_host_staging_bytes(p) >= need


def test_effective_k_follows_the_printed_formula(S):
    """stream_effective_k (host-only arithmetic inside the library) against hand values and the oracle."""
    from oracle import stream_oracle as so

    assert S.effective_k(1000, 32, 0.0) == 1
    assert S.effective_k(1000, 32, 1.0) == 31          # floor(T / b_q)
    assert S.effective_k(8192, 32, 0.1) == 26           # floor(1 + 255 * 0.1)
    assert S.effective_k(64, 64, 0.5) == 1
    for T in (1, 63, 64, 1000, 4096, 131072, 1048576):
        for bq in (1, 32, 64):
            for s in (0.0, 0.01, 0.04, 0.25, 0.5, 0.99, 1.0):
                assert S.stream_effective_k(T, bq, s) == so.effective_k(T, bq, s), (T, bq, s)
    for args in ((0, 32, 0.5), (100, 0, 0.5), (100, 32, -0.1), (100, 32, 1.01), (100, 32, float("nan"))):
        with pytest.raises(S.StreamError) as e:
            S.stream_effective_k(*args)
        assert e.value.status == S.STREAM_ERR_INVALID_ARG


def test_selftest_wait_rejects_bad_arguments_on_the_host(S):
    for limit in (0, -5, (1 << 31) + 1):
        with pytest.raises(S.StreamError) as e:
            S.stream_selftest_bounded_wait(limit, 256, 256, stream=0)
        assert e.value.status == S.STREAM_ERR_INVALID_ARG
    for ws, n in ((None, 256), (256, 128), (264, 256)):
        with pytest.raises(S.StreamError) as e:
            S.stream_selftest_bounded_wait(1000, ws, n, stream=0)
        assert e.value.status == S.STREAM_ERR_WORKSPACE


def test_unit_rate_probe_rejects_bad_arguments_on_the_host(S):
    lib = S._load()
    # no result record: refused before the device is even looked at
    assert lib.stream_probe_unit_rates(256, 1 << 30, None, None) == S.STREAM_ERR_INVALID_ARG
    out = S.StreamUnitRates()
    rc = lib.stream_probe_unit_rates(None, 0, ctypes.byref(out), None)
    assert rc in (S.STREAM_ERR_WORKSPACE, S.STREAM_ERR_CUDA)   # CUDA where there is no device to ask for its SM count
    assert S.stream_probe_scratch_bytes() % 256 == 0


@pytest.mark.parametrize("kw,s", [
    (dict(T=5000, k_top=9), 0.1), (dict(T=4096, k_top=32, causal=0), 0.3), (dict(T=777, block_q=16, block_k=16, d=64, k_top=5), 0.05),
    (dict(T=1000, block_q=32, block_k=8, d=64, k_top=12), 0.2), (dict(T=64, k_top=3), 0.9),
])
def test_k_schedule_is_host_only_and_matches_the_oracle(S, kw, s):
    """The per-row k schedule needs no GPU: checked here against the oracle's own formula."""
    import numpy as np
    import torch

    from oracle import stream_oracle as so

    p = good_problem(S, **kw)
    got = S.k_schedule(p, s)
    assert got.dtype == torch.int32 and not got.is_cuda
    op = so.OracleProblem(p.batch, p.n_q_heads, p.n_kv_heads, p.T, p.d, p.block_q, p.block_k, p.k_top, bool(p.causal), "bf16")
    np.testing.assert_array_equal(got.numpy(), so.k_schedule(op, s))
    assert got.min() >= 1 and got.max() <= p.k_top


def test_k_schedule_and_variable_k_reject_bad_arguments(S):
    import torch

    p = good_problem(S)
    out = torch.zeros(4, dtype=torch.int32)
    for s in (0.0, 1.0, -0.5, float("nan")):
        with pytest.raises(S.StreamError) as e:
            S.stream_k_schedule(p, s, out.data_ptr())
        assert e.value.status == S.STREAM_ERR_INVALID_ARG
    with pytest.raises(S.StreamError) as e:
        S.stream_k_schedule(p, 0.5, None)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
    with pytest.raises(S.StreamError) as e:  # a missing schedule is an error, not the fixed-k build
        S.stream_build_mask_var(p, 256, 256, None, 256, None, 256, 256, stream=0)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
