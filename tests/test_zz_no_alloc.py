"""alg_proj_forward_static -- the projection for callers that cannot allocate device memory
(a serving loop with a fixed memory pool, a plug-in whose host forbids cudaMalloc on the hot
path).  Its scratch is a fixed 8 MiB array inside the library, so the check here is simple: the
result must equal what alg_proj_forward produces with a caller-provided workspace, on two calls
in a row (the second call sees the scratch the first one left behind), and problems that do
not fit the array must be refused without launching anything.

Collected last on purpose (file name), so a run that stops at the first failure has already
run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _problem(M, seed, q=2, s_w=384, r_w=256):
    types = synth.uniform_types(500 + seed, M, q)
    return synth.make_workload("noalloc", config=6, variant=seed, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q,
                               types=types, integer=False, with_down=False)


def test_static_scratch_matches_workspace_entry_point_twice():
    proj = binding.Proj([384, 384], [256, 256], dtype="bf16")
    # Set-up call: the first use on a device looks up the address of the built-in array, which is
    # also when the driver places that part of the library image (8 MiB) on the GPU.  The checks
    # below are about the calls after it.
    wl0 = _problem(130, 9)
    proj.forward_static(H.to_dev(wl0.X, "bf16"), H.dev_types(wl0.types), H.to_dev(wl0.W_up, "bf16"),
                        torch.empty((130, 512), dtype=torch.float32, device="cuda"))
    for call, (M, seed) in enumerate([(700, 1), (333, 2)]):      # second call: other size, stale scratch
        wl = _problem(M, seed)
        X, t, W = H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16")
        want = proj.forward(X, t, W, act="gelu", out_dtype=torch.float32)
        got = torch.full_like(want, float("nan"))
        # Two witnesses that nothing was allocated.  torch's caching allocator served no request
        # (frees by the garbage collector do not touch that counter), and the device's free memory
        # as the driver reports it did not shrink -- the library links its own CUDA runtime, so a
        # cudaMalloc inside it would bypass torch's counter but not this one.
        torch.cuda.synchronize()
        before = torch.cuda.memory_stats()["allocation.all.allocated"]
        free_before = torch.cuda.mem_get_info()[0]
        proj.forward_static(X, t, W, got, act="gelu")
        torch.cuda.synchronize()
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == before
        assert torch.cuda.mem_get_info()[0] >= free_before
        assert proj.last_status() == 0
        # same kernels, same order of additions: the two entry points agree bit for bit,
        # which is tighter than the 5e-3 / 2e-2 bf16 tolerance the parity tests use
        assert torch.equal(got, want), f"call {call}"
        ref = np.vectorize(oracle.gelu)(oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))
        H.assert_bf16_close(H.to_np(got), ref, False, f"static scratch call {call}")


def test_static_scratch_fp32_path_and_size_limit():
    wl = synth.config1(integer=True)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="f32")
    X, t, W = H.to_dev(wl.X, "f32"), H.dev_types(wl.types), H.to_dev(wl.W_up, "f32")
    out = torch.empty((wl.M, wl.F), dtype=torch.float32, device="cuda")
    for _ in range(2):
        out.fill_(-1.0)
        proj.forward_static(X, t, W, out)
        assert torch.equal(out, proj.forward(X, t, W))
    # a bf16 problem whose bucketed copy of X alone exceeds the 8 MiB array is refused
    big = binding.Proj([2048, 2048], [256, 256], dtype="bf16")
    M = 4096
    assert big.workspace_bytes(M) > (8 << 20)
    Xb = torch.zeros((M, 4096), dtype=torch.bfloat16, device="cuda")
    Wb = torch.zeros((4096, 512), dtype=torch.bfloat16, device="cuda")
    tb = torch.zeros(M, dtype=torch.int32, device="cuda")
    ob = torch.full((M, 512), 3.0, dtype=torch.float32, device="cuda")
    launches = binding.launch_count()
    with pytest.raises(binding.AlgError) as e:
        big.forward_static(Xb, tb, Wb, ob)
    assert e.value.code == 3                      # ALG_ERR_WORKSPACE_TOO_SMALL
    assert binding.launch_count() == launches     # nothing was launched
    assert torch.all(ob == 3.0)
