"""GPU parity of the small-M (decode) kernel: M <= 64 rows, weights streamed once."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _wl(q, M, s_w, r_w, types=None, integer=True, seed=1):
    if types is None:
        types = synth.uniform_types(3000 + seed, M, q)
    return synth.make_workload("dec", config=4, variant=900 + seed, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q,
                               types=types, integer=integer, with_down=False)


@pytest.mark.parametrize("q,M,s_w,r_w", [
    (2, 1, 384, 1536), (2, 8, 384, 1536), (2, 33, 384, 1536), (2, 64, 384, 1536),   # up projection of config 4
    (2, 1, 1536, 384), (2, 17, 1536, 384), (2, 64, 1536, 384),                      # down projection of config 4
    (4, 5, 128, 512), (3, 64, 192, 128), (1, 16, 256, 256), (8, 40, 128, 128),
    (16, 40, 64, 128), (12, 9, 48, 64),   # more groups than the by-value table holds: table read from device memory
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_decode_integer_bit_exact(q, M, s_w, r_w, out_dtype):
    wl = _wl(q, M, s_w, r_w, seed=q * 100 + M)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    assert proj.kernel_path(M) == binding.ALG_PATH_DECODE
    Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype)
    assert proj.last_status() == 0
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first {bad[:5].tolist()}"


def test_decode_single_type_skips_unneeded_blocks():
    """All rows of one type: the other type's off-diagonal block is never read.  Poison it with
    NaNs -- the result must stay finite and exact."""
    q, M, s_w, r_w = 2, 8, 384, 1536
    wl = _wl(q, M, s_w, r_w, types=np.zeros(M, dtype=np.int32), seed=7)
    W = wl.W_up.copy()
    W[s_w:, :r_w] = np.nan          # W_10: used only by type-1 rows (x_1 W_10 enters y_0 of type-1 rows)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(W, "bf16"), out_dtype=torch.float32)
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    assert np.array_equal(H.to_np(Y), ref)


def test_decode_matches_prefill_kernel_and_oracle():
    """The same 64 rows through the decode kernel and, embedded in a larger batch, through the
    prefill kernels (same weights, same schedule) agree within the bf16 tolerance and both match
    the oracle."""
    q, s_w, r_w = 2, 384, 1536
    big = _wl(q, 640, s_w, r_w, integer=False, seed=11)
    proj = binding.Proj(big.d_widths, big.f_widths, dtype="bf16")
    Xd, td, Wd = H.to_dev(big.X, "bf16"), H.dev_types(big.types), H.to_dev(big.W_up, "bf16")
    bias = synth.bf16_round(synth.normal(77, (big.F,), 0.3))
    bd = H.to_dev(bias, "bf16")
    Y_pre = proj.forward(Xd, td, Wd, bias=bd, act="gelu", out_dtype=torch.float32)
    Y_dec = proj.forward(Xd[:64], td[:64], Wd, bias=bd, act="gelu", out_dtype=torch.float32)
    assert proj.kernel_path(640) == binding.ALG_PATH_TCGEN05 and proj.kernel_path(64) == binding.ALG_PATH_DECODE
    ref = np.vectorize(oracle.gelu)(oracle.proj(big.X[:64], big.types[:64], big.W_up, big.d_widths, big.f_widths, bias=bias))
    H.assert_bf16_close(H.to_np(Y_dec), ref, False, "decode")
    H.assert_bf16_close(H.to_np(Y_pre[:64]), ref, False, "prefill")
    assert H.max_abs(H.to_np(Y_dec), H.to_np(Y_pre[:64])) <= 1e-3


def test_decode_tables_cyclic_bad_type_and_determinism():
    q, M, s_w, r_w = 4, 24, 128, 256
    wl = _wl(q, M, s_w, r_w, seed=21)
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    dense = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", table="dense")
    assert np.array_equal(H.to_np(dense.forward(X, H.dev_types(wl.types), W, out_dtype=torch.float32)),
                          wl.X.astype(np.float64) @ wl.W_up.astype(np.float64))
    keep = oracle.support(4, "q2pow")
    cust = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", table="custom", custom_keep=torch.from_numpy(keep))
    assert np.array_equal(H.to_np(cust.forward(X, H.dev_types(wl.types), W, out_dtype=torch.float32)),
                          oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep))
    cyc = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    assert np.array_equal(H.to_np(cyc.forward(X, None, W, out_dtype=torch.float32)),
                          oracle.proj(wl.X, synth.cyclic_types(M, q), wl.W_up, wl.d_widths, wl.f_widths))
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    types = wl.types.copy()
    types[3] = 9
    Y1 = proj.forward(X, H.dev_types(types), W, out_dtype=torch.float32)
    assert proj.last_status() == 5
    Y2 = proj.forward(X, H.dev_types(types), W, out_dtype=torch.float32)
    assert torch.equal(Y1, Y2)
    got = H.to_np(Y1)
    assert not got[3].any()
    good = np.ones(M, bool)
    good[3] = False
    assert np.array_equal(got[good], oracle.proj(wl.X[good], types[good], wl.W_up, wl.d_widths, wl.f_widths))


def test_types_written_by_the_kernel_just_before():
    """The row types may be produced on the device right before the call (position mod q)."""
    q, M, s_w, r_w = 2, 24, 384, 1536
    wl = _wl(q, M, s_w, r_w, seed=31)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    pos = torch.from_numpy(np.arange(100, 100 + M, dtype=np.int32) * 3).cuda()
    buf = torch.zeros(M, dtype=torch.int32, device="cuda")
    out = torch.empty((M, wl.F), dtype=torch.float32, device="cuda")
    for rep in range(3):
        buf.zero_()                               # stale contents the early read may see
        torch.remainder(pos + rep, q, out=buf)    # the types of this step, written just before the call
        proj.forward(X, buf, W, out=out)
        t = ((np.arange(100, 100 + M) * 3 + rep) % q).astype(np.int32)
        assert np.array_equal(H.to_np(out), oracle.proj(wl.X, t, wl.W_up, wl.d_widths, wl.f_widths)), rep
    assert proj.last_status() == 0


def test_bounded_wait_expires_and_the_handle_recovers():
    """A device-side wait that cannot complete must end by itself: the status word reports
    ALG_ERR_DEVICE_TIMEOUT, the call returns, and the same handle computes exactly again
    afterwards.  The stall is made without any fault: the kernel is told to expect 1 KiB more on
    its weight barrier than its copies deliver (every issued copy still lands), with the wait
    limit lowered to a few milliseconds."""
    q, M, s_w, r_w = 2, 8, 384, 1536
    wl = _wl(q, M, s_w, r_w, seed=41)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    X, t, W = H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16")
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    assert np.array_equal(H.to_np(proj.forward(X, t, W, out_dtype=torch.float32)), ref)
    proj.set_option("wait_limit_cycles", 8_000_000)      # about 4 ms
    proj.set_option("test_stall_bytes", 1024)
    proj.forward(X, t, W, out_dtype=torch.float32)
    assert proj.last_status() == 6                        # ALG_ERR_DEVICE_TIMEOUT, and the call came back
    assert proj.last_status() == 0                        # reading cleared it
    proj.set_option("test_stall_bytes", 0)
    proj.set_option("wait_limit_cycles", 4_000_000_000)
    assert np.array_equal(H.to_np(proj.forward(X, t, W, out_dtype=torch.float32)), ref)
    assert proj.last_status() == 0
