"""The allocation-free mask entry point against the workspace one.

Some users of the library cannot allocate device memory when they call it (their process gave
all of HBM to its own pool at start-up, or they sit in a loop that must not stall on cudaMalloc's
implicit synchronisation). stream_build_mask_static serves them from a scratch array built into
the library. This file is collected last on purpose, and must pass both alone and after the rest.
"""
import pytest
import torch

from paper_2510_19875_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    from paper_2510_19875_b200 import stream as S

    specs = [
        wl.WorkloadSpec("na1", 31, 1, 8, 2, 8192, 128, 64, 16, "bf16", sink=True, anchors=True),  # tensor-core kernel
        wl.WorkloadSpec("na2", 32, 2, 2, 1, 1000, 64, 32, 5, "f32"),                              # generic kernel
    ]
    for spec in specs:  # two calls in a row on the shared scratch, different shapes and kernels
        w = wl.generate(spec, with_v=False)
        q, k, _ = w.torch_tensors("cuda")
        ref = S.build_mask(q, k, block_q=spec.block, block_k=spec.block, k_top=spec.k_top, want_scores=True)
        p = S.make_problem(q, k, block_q=spec.block, block_k=spec.block, k_top=spec.k_top)
        for _ in range(2):
            mask = torch.full_like(ref.mask, -7)
            scores = torch.zeros_like(ref.scores)
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated()
            # the driver's own count of free bytes sees what torch's allocator cannot: a cudaMalloc
            # inside the library. (The kernels' code was loaded by the workspace calls above.)
            free_before = torch.cuda.mem_get_info()[0]
            S.stream_build_mask_static(p, q, k, mask, scores)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] >= free_before
            assert torch.equal(mask, ref.mask)       # masks are integer work: bit-exact
            assert torch.equal(scores, ref.scores)   # same kernel, same inputs: same fp32 scores


def test_static_scratch_entry_point_validates_like_the_other():
    from paper_2510_19875_b200 import stream as S

    q = torch.zeros(1, 2, 128, 64, device="cuda")
    p = S.make_problem(q, q, block_q=32, block_k=32, k_top=2)
    p.k_top = 0
    with pytest.raises(S.StreamError) as e:
        S.stream_build_mask_static(p, q, q, q, None)
    assert e.value.status == S.STREAM_ERR_INVALID_ARG
    # a valid request that no kernel covers: the same status from both entry points
    p = S.make_problem(q, q, block_q=32, block_k=32, k_top=2)
    p.k_top = 2000
    ws = torch.empty(256, dtype=torch.uint8, device="cuda")
    for call in (lambda: S.stream_build_mask_static(p, q, q, q, None),
                 lambda: S.stream_build_mask(p, q, q, q, None, ws, ws.numel())):
        with pytest.raises(S.StreamError) as e:
            call()
        assert e.value.status == S.STREAM_ERR_UNSUPPORTED
