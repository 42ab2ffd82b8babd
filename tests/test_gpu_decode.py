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


# ---- the decode step of the whole FFN in one launch (M <= 16) -----------------------------------

def _ffn_int_workload(q, M, D, F, types=None, seed=1):
    """Integer FFN problem whose hidden state stays exactly representable in bf16 (entries of X and
    W_down in {-1,0,1}, W_up sparse), so that with act = none both projections are exact."""
    if types is None:
        types = synth.uniform_types(4000 + seed, M, q)
    wl = synth.make_workload("ffndec", config=4, variant=700 + seed, dtype="bf16", q=q, M=M, D=D, F=F, types=types,
                             integer=True)
    wl.X = np.sign(wl.X).astype(np.float32)
    wl.W_up = (np.sign(wl.W_up) * (np.abs(wl.W_up) > 2)).astype(np.float32)
    wl.W_down = np.sign(wl.W_down).astype(np.float32)
    return wl


def _ffn_int_ref(wl, keep=None, b_up=None, b_down=None):
    Hh = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep, bias=b_up)
    assert np.abs(Hh).max() <= 256          # exactly representable in bf16
    return oracle.proj(Hh, wl.types, wl.W_down, wl.f_widths, wl.d_widths, keep=keep, bias=b_down)


@pytest.mark.parametrize("q,M,D,F", [
    (2, 1, 768, 3072), (2, 3, 768, 3072), (2, 8, 768, 3072), (2, 9, 768, 3072), (2, 16, 768, 3072),   # config 4
    (4, 5, 512, 2048), (3, 16, 192, 384), (1, 7, 256, 512), (8, 12, 512, 1024),
    (16, 11, 1024, 2048),      # table read from device memory
    (2, 16, 96, 160),          # widths that are no multiples of 64: ragged last K chunk
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_ffn_decode_one_launch_integer_bit_exact(q, M, D, F, out_dtype):
    wl = _ffn_int_workload(q, M, D, F, seed=q * 50 + M)
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
    bu = synth.small_ints(71, (F,), -2, 2)
    bd = synth.small_ints(72, (D,), -2, 2)
    args = (H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"))
    launches = binding.launch_count()
    Y = ffn.forward(*args, b_up=H.to_dev(bu, "bf16"), b_down=H.to_dev(bd, "bf16"), act=None, out_dtype=out_dtype)
    assert binding.launch_count() - launches == 1          # one kernel for the whole FFN
    assert ffn.last_status() == 0
    ref = _ffn_int_ref(wl, b_up=bu, b_down=bd)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first {bad[:5].tolist()}"
    # the two-kernel path of the same handle gives the same bits
    ffn.set_option("small_m_kernel", 0)
    Y2 = ffn.forward(*args, b_up=H.to_dev(bu, "bf16"), b_down=H.to_dev(bd, "bf16"), act=None, out_dtype=out_dtype)
    assert np.array_equal(H.to_np(Y2), ref)


def test_ffn_decode_skips_blocks_no_row_needs():
    """All rows of type 0: W_10 of both banks is used by nobody.  Poisoned with NaN it must stay
    unread; the same for type 1 and W_01."""
    q, M, D, F = 2, 6, 768, 3072
    for t in (0, 1):
        wl = _ffn_int_workload(q, M, D, F, types=np.full(M, t, dtype=np.int32), seed=90 + t)
        Wu, Wd = wl.W_up.copy(), wl.W_down.copy()
        o = 1 - t   # block (o, t): input group o, output group t is needed only by rows of type o
        Wu[o * 384:(o + 1) * 384, t * 1536:(t + 1) * 1536] = np.nan
        Wd[o * 1536:(o + 1) * 1536, t * 384:(t + 1) * 384] = np.nan
        ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
        Y = ffn.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(Wu, "bf16"), H.to_dev(Wd, "bf16"),
                        act=None, out_dtype=torch.float32)
        assert np.array_equal(H.to_np(Y), _ffn_int_ref(wl)), t


def test_ffn_decode_tables_cyclic_bad_type_gelu():
    q, M, D, F = 4, 13, 512, 1024
    wl = _ffn_int_workload(q, M, D, F, seed=7)
    X, Wu, Wd = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16")
    for table in ("dense", "q2pow"):
        keep = oracle.support(q, table)
        ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", table=table)
        Y = ffn.forward(X, H.dev_types(wl.types), Wu, Wd, act=None, out_dtype=torch.float32)
        assert np.array_equal(H.to_np(Y), _ffn_int_ref(wl, keep=keep)), table
    cyc = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    wc = _ffn_int_workload(q, M, D, F, types=synth.cyclic_types(M, q), seed=7)
    Y = cyc.forward(X, None, Wu, Wd, act=None, out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), _ffn_int_ref(wc))
    # out-of-range types: status, zero rows, the other rows exact; bitwise repeatable
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
    types = wl.types.copy()
    types[[2, 12]] = [7, -1]
    Y1 = ffn.forward(X, H.dev_types(types), Wu, Wd, act=None, out_dtype=torch.float32)
    assert ffn.last_status() == 5
    Y2 = ffn.forward(X, H.dev_types(types), Wu, Wd, act=None, out_dtype=torch.float32)
    assert torch.equal(Y1, Y2)
    got = H.to_np(Y1)
    assert not got[[2, 12]].any()
    good = np.ones(M, bool)
    good[[2, 12]] = False
    assert np.array_equal(got[good], _ffn_int_ref(wl)[good])
    # real-valued data with GELU and biases against the fp64 oracle
    w = synth.make_workload("ffndec-n", config=4, variant=777, dtype="bf16", q=2, M=16, D=768, F=3072,
                            types=synth.decode_types(5, 16, 2))
    bu, bd = synth.bf16_round(synth.normal(8, (w.F,), 0.2)), synth.bf16_round(synth.normal(9, (w.D,), 0.2))
    f2 = binding.FFN(w.d_widths, w.f_widths, dtype="bf16")
    Yn = f2.forward(H.to_dev(w.X, "bf16"), H.dev_types(w.types), H.to_dev(w.W_up, "bf16"), H.to_dev(w.W_down, "bf16"),
                    b_up=H.to_dev(bu, "bf16"), b_down=H.to_dev(bd, "bf16"), act="gelu", out_dtype=torch.float32)
    ref = oracle.ffn(w.X, w.types, w.W_up, w.W_down, w.d_widths, w.f_widths, b_up=bu, b_down=bd)
    H.assert_bf16_close(H.to_np(Yn), ref, False, "one-launch decode FFN")


def test_ffn_decode_chain_in_a_graph_replays():
    """Six dependent layers (distinct weights, layer l+1 reads layer l's output) captured in one
    CUDA graph, as the streaming benchmark does: consecutive launches overlap through programmatic
    dependent launch and share the handle's exchange counters.  Every replay must reproduce, bit
    for bit, the result of running the layers one at a time with a device synchronisation between
    them; that result is checked against the oracle layer by layer."""
    q, M, D, F, L = 2, 8, 768, 3072, 6
    wl = synth.config4(M)
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
    t = H.dev_types(wl.types)
    Wu_h = [synth.bf16_round(synth.normal(100 + l, (D, F), 0.02)) for l in range(L)]
    Wd_h = [synth.bf16_round(synth.normal(200 + l, (F, D), 0.02)) for l in range(L)]
    Wu, Wd = [H.to_dev(w, "bf16") for w in Wu_h], [H.to_dev(w, "bf16") for w in Wd_h]
    acts = [H.to_dev(wl.X, "bf16")] + [torch.zeros((M, D), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    ws = torch.empty(ffn.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    want = [acts[0]]
    for l in range(L):       # one layer at a time
        want.append(ffn.forward(want[l], t, Wu[l], Wd[l], act="gelu", workspace=ws))
        torch.cuda.synchronize()
        ref = oracle.ffn(H.to_np(want[l]), wl.types, Wu_h[l], Wd_h[l], wl.d_widths, wl.f_widths)
        H.assert_bf16_close(H.to_np(want[l + 1]), ref, True, f"layer {l}")
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        for l in range(L):   # back to back, overlapping
            ffn.forward(acts[l], t, Wu[l], Wd[l], act="gelu", out=acts[l + 1], workspace=ws, stream=stream)
        stream.synchronize()
        for l in range(L):
            assert torch.equal(acts[l + 1], want[l + 1]), f"eager layer {l}"
        with torch.cuda.graph(g, stream=stream):
            for l in range(L):
                ffn.forward(acts[l], t, Wu[l], Wd[l], act="gelu", out=acts[l + 1], workspace=ws, stream=stream)
    for rep in range(4):
        for l in range(L):
            acts[l + 1].zero_()
        g.replay()
        torch.cuda.synchronize()
        for l in range(L):
            assert torch.equal(acts[l + 1], want[l + 1]), f"replay {rep} layer {l}"
    assert ffn.last_status() == 0


def test_ffn_decode_bounded_waits_expire_and_the_handle_recovers():
    q, M, D, F = 2, 4, 768, 3072
    wl = _ffn_int_workload(q, M, D, F, seed=55)
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
    args = (H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"))
    ref = _ffn_int_ref(wl)
    assert np.array_equal(H.to_np(ffn.forward(*args, act=None, out_dtype=torch.float32)), ref)
    ffn.set_option("wait_limit_cycles", 6_000_000)       # about 3 ms per wait
    ffn.set_option("test_stall_bytes", 512)
    ffn.forward(*args, act=None, out_dtype=torch.float32)
    assert ffn.last_status() == 6                         # the weight barrier and then the exchange gave up
    ffn.set_option("test_stall_bytes", 0)
    ffn.set_option("wait_limit_cycles", 4_000_000_000)
    for _ in range(2):                                    # counters were reset with the status
        assert np.array_equal(H.to_np(ffn.forward(*args, act=None, out_dtype=torch.float32)), ref)
    assert ffn.last_status() == 0


# ---- one row (M = 1) under the complete-graph law with equal groups: one launch of plain FMAs ----------------

@pytest.mark.parametrize("q,s_w,r_w", [
    (32, 64, 192), (32, 80, 304), (32, 128, 384), (32, 64, 24), (32, 224, 64),   # the public shapes of the paper's kernel tables
    (64, 40, 200),      # an algebra beyond 32 groups (large-algebra handle)
    (5, 24, 40),        # pieces of 8 columns on both sides
    (1, 256, 512),      # q = 1: an ordinary matrix-vector product
])
def test_one_row_projection_in_one_launch(q, s_w, r_w):
    """A projection of one row: one launch, integers exact against the oracle for both output types, bias and GELU
    within the bf16 tolerance."""
    wl = _wl(q, 1, s_w, r_w, types=np.array([(3 * q) // 4 % q], np.int32), seed=q + s_w)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    assert proj.kernel_path(1) == binding.ALG_PATH_DECODE
    X, t, W = H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16")
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    for out_dtype in (torch.float32, torch.bfloat16):
        n0 = binding.launch_count()
        Y = proj.forward(X, t, W, out_dtype=out_dtype)
        assert binding.launch_count() - n0 == 1 and proj.last_status() == 0
        assert np.array_equal(H.to_np(Y), ref if out_dtype == torch.float32 else H.bf16_rne(ref))
    wr = _wl(q, 1, s_w, r_w, types=wl.types, integer=False, seed=q + s_w + 1)
    bias = synth.bf16_round(synth.normal(6, (wr.F,), 0.5))
    Xr, Wr = H.to_dev(wr.X, "bf16"), H.to_dev(wr.W_up, "bf16")
    for act in (None, "gelu", "gelu_tanh"):
        Y = proj.forward(Xr, t, Wr, bias=H.to_dev(bias, "bf16"), act=act, out_dtype=torch.float32)
        z = oracle.proj(wr.X, wr.types, wr.W_up, wr.d_widths, wr.f_widths, bias=bias)
        if act == "gelu":
            z = np.vectorize(oracle.gelu)(z)
        elif act == "gelu_tanh":
            z = 0.5 * z * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (z + 0.044715 * z ** 3)))
        H.assert_bf16_close(H.to_np(Y), z, False, f"one row act={act}")


def test_one_row_type_written_just_before_and_out_of_range():
    """The kernel reads the row type before its launch dependency resolves (to request weights early) and again
    after: a type written on the device right before the call is the one that counts.  A type outside [0, q) gives a
    zero row and status 5."""
    q, s_w, r_w = 8, 64, 128
    wl = _wl(q, 1, s_w, r_w, seed=77)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    buf = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.empty((1, wl.F), dtype=torch.float32, device="cuda")
    for rep in range(5):
        buf.fill_((rep * 5) % q)                  # stale: what the early read may see
        buf.fill_((rep * 3 + 1) % q)              # the type of this step, written just before the call
        proj.forward(X, buf, W, out=out)
        t = np.array([(rep * 3 + 1) % q], np.int32)
        assert np.array_equal(H.to_np(out), oracle.proj(wl.X, t, wl.W_up, wl.d_widths, wl.f_widths)), rep
    assert proj.last_status() == 0
    buf.fill_(q)
    out.fill_(7.0)
    proj.forward(X, buf, W, out=out)
    assert proj.last_status() == 5 and np.all(H.to_np(out) == 0)


@pytest.mark.parametrize("q,D,F", [(32, 4096, 12288), (32, 2048, 768), (4, 256, 1024)])
def test_one_row_ffn_in_one_launch(q, D, F):
    """FFN shapes the staged one-launch decode kernel does not hold in shared memory: one row is two matrix-vector
    phases around a bounded wait, biases and GELU included; twice in a row (the counters are cleared by the kernel)."""
    types = np.array([q // 2], np.int32)
    wl = synth.make_workload("ffnrow", config=4, variant=q + D, dtype="bf16", q=q, M=1, D=D, F=F, types=types)
    wl.W_up, wl.W_down = synth.bf16_round(wl.W_up * 2.0), synth.bf16_round(wl.W_down * 2.0)
    b_up = synth.bf16_round(synth.normal(8, (F,), 0.3))
    b_down = synth.bf16_round(synth.normal(9, (D,), 0.3))
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
    args = (H.to_dev(wl.X, "bf16"), H.dev_types(types), H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"))
    ref = oracle.ffn(wl.X, types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, b_up=b_up, b_down=b_down)
    for out_dtype in (torch.float32, torch.bfloat16):
        n0 = binding.launch_count()
        Y = ffn.forward(*args, b_up=H.to_dev(b_up, "bf16"), b_down=H.to_dev(b_down, "bf16"), act="gelu", out_dtype=out_dtype)
        assert binding.launch_count() - n0 == 1 and ffn.last_status() == 0
        H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"one-row FFN q={q}")


@pytest.mark.parametrize("k", range(18))
def test_one_row_random_shapes(k):
    """Random group counts and widths for the one-row kernel: projection (integers exact), FFN and gated FFN (tolerance)."""
    rng = np.random.default_rng(52000 + k)
    q = int(rng.choice([1, 2, 3, 5, 8, 16, 32, 40, 64, 100, 256]))
    s_w = 8 * int(rng.integers(1, 20 if q <= 40 else 5))
    r_w = 8 * int(rng.integers(1, 40 if q <= 40 else 9))
    t = np.array([int(rng.integers(0, q))], np.int32)
    mode = k % 3 if q <= 32 else 0
    if mode == 0:
        wl = _wl(q, 1, s_w, r_w, types=t, seed=k)
        proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
        Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(t), H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
        assert proj.last_status() == 0
        assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, t, wl.W_up, wl.d_widths, wl.f_widths))
    elif mode == 1:
        wl = synth.make_workload("row1", config=4, variant=k, dtype="bf16", q=q, M=1, D=s_w * q, F=r_w * q, types=t)
        ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16")
        Y = ffn.forward(H.to_dev(wl.X, "bf16"), H.dev_types(t), H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"),
                        act="gelu", out_dtype=torch.float32)
        assert ffn.last_status() == 0
        H.assert_bf16_close(H.to_np(Y), oracle.ffn(wl.X, t, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths), False, f"one-row FFN {k}")
    else:
        wl, Wg = synth.gated_ffn("row1g", q, 1, s_w * q, r_w * q, t, variant=k)
        ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16")
        Y = ffn.forward(H.to_dev(wl.X, "bf16"), H.dev_types(t), H.to_dev(np.concatenate([Wg, wl.W_up], axis=1), "bf16"),
                        H.to_dev(wl.W_down, "bf16"), out_dtype=torch.float32)
        assert ffn.last_status() == 0
        H.assert_bf16_close(H.to_np(Y), oracle.ffn_swiglu(wl.X, t, Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths), False,
                            f"one-row gated FFN {k}")


@pytest.mark.parametrize("q,s_w,r_w", [(32, 64, 192), (32, 128, 384), (5, 24, 40), (64, 40, 200)])
@pytest.mark.parametrize("M", [2, 5, 8])
def test_few_rows_on_the_row_kernel(q, s_w, r_w, M):
    """Up to eight rows on the row kernel (forced with SMALL_M_KERNEL = 3; by its own choice the library takes it while
    the rows' weight segments stay below the measured break-even): projection exact on integers, FFN and gated FFN within
    tolerance, explicit and cyclic types, one launch each."""
    for schedule in ("explicit", "cyclic"):
        types = synth.cyclic_types(M, q) if schedule == "cyclic" else synth.uniform_types(5000 + q + M, M, q)
        t = None if schedule == "cyclic" else H.dev_types(types)
        wl = _wl(q, M, s_w, r_w, types=types, seed=q + M)
        proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
        proj.set_option("small_m_kernel", 3)
        n0 = binding.launch_count()
        Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
        assert binding.launch_count() - n0 == 1 and proj.last_status() == 0
        assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, types, wl.W_up, wl.d_widths, wl.f_widths))
        if q > 32:
            continue
        wf = synth.make_workload("rows-ffn", config=4, variant=q + M, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q, types=types)
        ffn = binding.FFN(wf.d_widths, wf.f_widths, dtype="bf16", schedule=schedule)
        ffn.set_option("small_m_kernel", 3)
        n0 = binding.launch_count()
        Y = ffn.forward(H.to_dev(wf.X, "bf16"), t, H.to_dev(wf.W_up, "bf16"), H.to_dev(wf.W_down, "bf16"), act="gelu",
                        out_dtype=torch.bfloat16)
        assert binding.launch_count() - n0 == 1 and ffn.last_status() == 0
        H.assert_bf16_close(H.to_np(Y), oracle.ffn(wf.X, types, wf.W_up, wf.W_down, wf.d_widths, wf.f_widths), True, "rows FFN")
        wg, Wg = synth.gated_ffn("rows-gated", q, M, s_w * q, r_w * q, types, variant=q + M)
        gf = binding.GatedFFN(wg.d_widths, wg.f_widths, dtype="bf16", schedule=schedule)
        gf.set_option("small_m_kernel", 3)
        n0 = binding.launch_count()
        Y = gf.forward(H.to_dev(wg.X, "bf16"), t, H.to_dev(np.concatenate([Wg, wg.W_up], axis=1), "bf16"), H.to_dev(wg.W_down, "bf16"),
                       out_dtype=torch.float32)
        assert binding.launch_count() - n0 == 1 and gf.last_status() == 0
        H.assert_bf16_close(H.to_np(Y), oracle.ffn_swiglu(wg.X, types, Wg, wg.W_up, wg.W_down, wg.d_widths, wg.f_widths), False,
                            "rows gated FFN")


def test_few_rows_one_type_out_of_range_and_types_written_just_before():
    q, s_w, r_w, M = 8, 64, 128, 6
    wl = _wl(q, M, s_w, r_w, seed=91)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    proj.set_option("small_m_kernel", 3)
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    buf = torch.zeros(M, dtype=torch.int32, device="cuda")
    out = torch.empty((M, wl.F), dtype=torch.float32, device="cuda")
    pos = torch.arange(M, dtype=torch.int32, device="cuda")
    for rep in range(4):
        buf.fill_(rep % q)                                  # stale: what the early read may see
        torch.remainder(pos * 3 + rep, q, out=buf)          # the types of this step, written just before the call
        proj.forward(X, buf, W, out=out)
        t = ((np.arange(M) * 3 + rep) % q).astype(np.int32)
        assert np.array_equal(H.to_np(out), oracle.proj(wl.X, t, wl.W_up, wl.d_widths, wl.f_widths)), rep
    assert proj.last_status() == 0
    t = np.array([1, 2, q + 3, 0, -1, 5], np.int32)
    out.fill_(7.0)
    proj.forward(X, H.dev_types(t), W, out=out)
    assert proj.last_status() == 5
    got = H.to_np(out)
    good = [0, 1, 3, 5]
    assert np.all(got[[2, 4]] == 0)
    assert np.array_equal(got[good], oracle.proj(wl.X[good], t[good], wl.W_up, wl.d_widths, wl.f_widths))
