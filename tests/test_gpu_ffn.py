"""GPU parity of alg_ffn_forward (up -> GELU -> down) against the fp64 oracle, at the benchmark
configurations (or the rows the oracle can afford) and on edge cases."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _ffn(wl, table="qq", schedule="explicit", custom=None):
    return binding.FFN(wl.d_widths, wl.f_widths, dtype=wl.dtype, table=table, schedule=schedule, custom_keep=custom)


def _run_ffn(wl, ffn, out_dtype, b_up=None, b_down=None, act="gelu", types=True):
    X = H.to_dev(wl.X, wl.dtype)
    Wu, Wd = H.to_dev(wl.W_up, wl.dtype), H.to_dev(wl.W_down, wl.dtype)
    bu = None if b_up is None else H.to_dev(b_up, wl.dtype)
    bd = None if b_down is None else H.to_dev(b_down, wl.dtype)
    Y = ffn.forward(X, H.dev_types(wl.types) if types else None, Wu, Wd, b_up=bu, b_down=bd, act=act,
                    out_dtype=out_dtype)
    assert ffn.last_status() == 0
    return Y


def _sample_rows(wl, per_type, seed=0):
    """first/last rows of every bucket, rows inside the ragged last tile, plus random rows."""
    rng = np.random.default_rng(seed)
    rows = []
    for t in range(wl.q):
        idx = np.flatnonzero(wl.types == t)
        if idx.size == 0:
            continue
        tail = idx[(idx.size // 128) * 128:]
        pick = np.concatenate([idx[:2], idx[-2:], tail[:2], rng.choice(idx, size=min(per_type, idx.size), replace=False)])
        rows.append(pick)
    return np.unique(np.concatenate(rows))


def test_ffn_f32_simt_small():
    wl = synth.make_workload("ffn32", config=7, variant=1, dtype="f32", q=3, M=200, D=96, F=240,
                             types=synth.uniform_types(3, 200, 3), x_std=1.0, w_std=0.1)
    bu, bd = synth.normal(11, (wl.F,), 0.1), synth.normal(12, (wl.D,), 0.1)
    Y = _run_ffn(wl, _ffn(wl), torch.float32, b_up=bu, b_down=bd)
    ref = oracle.ffn(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, b_up=bu, b_down=bd)
    got = H.to_np(Y)
    assert H.rel_fro(got, ref) <= 1e-5 and H.max_abs(got, ref) <= 1e-4


@pytest.mark.parametrize("kernel", [0, 1, 4])   # the library's choice, the table-driven kernel, the large-algebra kernel
def test_ffn_integer_identity_activation_bit_exact(kernel):
    """With act = none both projections are exact integer arithmetic through the tensor cores
    (|H| <= 9*256 stays exactly representable in bf16 only if small: use entries in {-1,0,1})."""
    wl = synth.make_workload("ffnint", config=7, variant=2, dtype="bf16", q=2, M=600, D=128, F=256,
                             types=synth.uniform_types(4, 600, 2), integer=True)
    wl.X = np.sign(wl.X).astype(np.float32)
    wl.W_up = np.sign(wl.W_up).astype(np.float32) * (np.abs(wl.W_up) > 2)
    wl.W_down = np.sign(wl.W_down).astype(np.float32)
    ffn = _ffn(wl)
    ffn.set_option("gemm_kernel", kernel)
    Y = _run_ffn(wl, ffn, torch.float32, act=None)
    Hh = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    assert np.abs(Hh).max() <= 256  # exactly representable in bf16
    ref = oracle.proj(Hh, wl.types, wl.W_down, wl.f_widths, wl.d_widths)
    assert np.array_equal(H.to_np(Y), ref)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_cfg2_full_every_output(out_dtype):
    wl = synth.config2()
    ffn = _ffn(wl)
    Y = _run_ffn(wl, ffn, out_dtype)
    rows = np.arange(0, wl.M, 4) if out_dtype == torch.bfloat16 else np.arange(wl.M)
    ref = oracle.ffn(wl.X[rows], wl.types[rows], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y)[rows], ref, out_dtype == torch.bfloat16, "cfg2")
    assert ffn.macs([4096, 4096]) == 2 * 8192 * 768 * 3072 * 3 // 4


def test_cfg2_cyclic_schedule_and_dense_control():
    wl = synth.config2(M=2048)
    Y = _run_ffn(wl, _ffn(wl, schedule="cyclic"), torch.float32, types=False)
    ref = oracle.ffn(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y), ref, False, "cfg2 cyclic")
    Yd = _run_ffn(wl, _ffn(wl, table="dense"), torch.float32)
    refd = oracle.ffn(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=oracle.support(2, "dense"))
    H.assert_bf16_close(H.to_np(Yd), refd, False, "cfg2 dense control")


@pytest.mark.parametrize("q", [4, 8])
def test_cfg3_full_size_sampled_rows(q):
    wl = synth.config3(q)
    ffn = _ffn(wl)
    Y = _run_ffn(wl, ffn, torch.float32)
    rows = _sample_rows(wl, 192, seed=q)
    ref = oracle.ffn(wl.X[rows], wl.types[rows], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y[torch.from_numpy(rows).cuda()]), ref, False, f"cfg3 q={q}")
    if q == 4:   # the same launch with bf16 output: final rounding adds half an ulp to the bound
        Yb = _run_ffn(wl, ffn, torch.bfloat16)
        H.assert_bf16_close(H.to_np(Yb[torch.from_numpy(rows).cuda()]), ref, True, f"cfg3 q={q} bf16 out")
    # the square d -> d projection of the same configuration
    proj = binding.Proj(wl.d_widths, wl.d_widths, dtype="bf16")
    Wsq = synth.bf16_round(synth.normal(synth.seed_for(3, q) + 9, (wl.D, wl.D), 0.02))
    Ysq = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(Wsq, "bf16"), out_dtype=torch.float32)
    refsq = oracle.proj(wl.X[rows], wl.types[rows], Wsq, wl.d_widths, wl.d_widths)
    H.assert_bf16_close(H.to_np(Ysq[torch.from_numpy(rows).cuda()]), refsq, False, f"cfg3 square q={q}")


@pytest.mark.parametrize("M", [1, 8, 32, 64])
def test_cfg4_decode_shapes(M):
    wl = synth.config4(M)
    Y = _run_ffn(wl, _ffn(wl), torch.float32)
    ref = oracle.ffn(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y), ref, False, f"cfg4 M={M}")
    Yb = _run_ffn(wl, _ffn(wl), torch.bfloat16)
    H.assert_bf16_close(H.to_np(Yb), ref, True, f"cfg4 M={M} bf16 out")


@pytest.mark.parametrize("q", [2, 4, 8, 16])
def test_cfg5_full_size_sampled_rows(q):
    """Full-size launch (the configuration the benchmark times); the oracle checks every output
    of >= 64 sampled rows per type, including bucket ends and ragged-tile rows."""
    wl = synth.config5(q)
    ffn = _ffn(wl)
    Y = _run_ffn(wl, ffn, torch.float32)
    rows = _sample_rows(wl, 64, seed=q)
    assert all((wl.types[rows] == t).sum() >= 64 for t in range(q))
    ref = oracle.ffn(wl.X[rows], wl.types[rows], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y[torch.from_numpy(rows).cuda()]), ref, False, f"cfg5 q={q}")
    # plus 4096 single outputs at random (row, column) positions of the whole result
    rng = np.random.default_rng(500 + q)
    er, ec = rng.integers(0, wl.M, size=4096), rng.integers(0, wl.D, size=4096)
    want = oracle.ffn_entries(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, er, ec)
    got = Y[torch.from_numpy(er).cuda(), torch.from_numpy(ec).cuda()].double().cpu().numpy()
    H.assert_bf16_close(got, want, False, f"cfg5 q={q} single entries")
    if q == 8:   # the same launch with bf16 output
        del Y
        Yb = _run_ffn(wl, ffn, torch.bfloat16)
        H.assert_bf16_close(H.to_np(Yb[torch.from_numpy(rows).cuda()]), ref, True, f"cfg5 q={q} bf16 out")
        got = Yb[torch.from_numpy(er).cuda(), torch.from_numpy(ec).cuda()].double().cpu().numpy()
        H.assert_bf16_close(got, want, True, f"cfg5 q={q} single entries, bf16 out")
        del Yb
    else:
        del Y
    torch.cuda.empty_cache()


def test_ffn_host_entry_point_matches_device_entry_point():
    wl = synth.config2(M=1024)
    ffn = _ffn(wl)
    Yd = _run_ffn(wl, ffn, torch.float32)
    Xh = torch.from_numpy(wl.X).to(torch.bfloat16).pin_memory()
    th = torch.from_numpy(wl.types).pin_memory()
    Yh = torch.empty((wl.M, wl.D), dtype=torch.float32).pin_memory()
    ffn.forward_host(Xh, th, H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"), Yh)
    torch.cuda.synchronize()
    assert torch.equal(Yh, Yd.cpu())


def test_ffn_graph_capture_replays():
    wl = synth.config2(M=1024)
    ffn = _ffn(wl)
    X, t = H.to_dev(wl.X, "bf16"), H.dev_types(wl.types)
    Wu, Wd = H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16")
    Y = torch.zeros((wl.M, wl.D), dtype=torch.float32, device="cuda")
    ws = torch.empty(ffn.workspace_bytes(wl.M), dtype=torch.uint8, device="cuda")
    ffn.forward(X, t, Wu, Wd, out=Y, workspace=ws)
    want = Y.clone()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        ffn.forward(X, t, Wu, Wd, out=Y, workspace=ws, stream=s)   # warm-up on the capture stream
        with torch.cuda.graph(g, stream=s):
            ffn.forward(X, t, Wu, Wd, out=Y, workspace=ws, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    for _ in range(3):
        Y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(Y, want)


@pytest.mark.parametrize("q,M", [(2, 1024), (4, 1000), (4, 1001), (3, 771)])
def test_cyclic_fast_path_matches_explicit_types(q, M):
    """type = row mod q.  When q divides M the library skips bucketing and gathering (type-strided
    tensor map, arithmetic row scatter); otherwise it takes the general path.  On one kernel both must equal
    the explicit-types result bit for bit (the kernels differ in the order of their sums, so the library's own
    choices -- which may differ between the two schedules -- are compared with the oracle), and the oracle
    within tolerance."""
    wl = synth.make_workload("cyc", config=7, variant=q * 1000 + M, dtype="bf16", q=q, M=M, D=q * 128, F=q * 256,
                             types=synth.cyclic_types(M, q))
    ref = oracle.ffn(wl.X, wl.types, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    for kernel in (1, 4, 0):
        f_exp, f_cyc = _ffn(wl), _ffn(wl, schedule="cyclic")
        f_exp.set_option("gemm_kernel", kernel)
        f_cyc.set_option("gemm_kernel", kernel)
        Y_exp = _run_ffn(wl, f_exp, torch.float32)
        Y_cyc = _run_ffn(wl, f_cyc, torch.float32, types=False)
        if kernel:
            assert torch.equal(Y_exp, Y_cyc), kernel
        H.assert_bf16_close(H.to_np(Y_exp), ref, False, f"explicit q={q} M={M} kernel={kernel}")
        H.assert_bf16_close(H.to_np(Y_cyc), ref, False, f"cyclic q={q} M={M} kernel={kernel}")
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    Yp = proj.forward(H.to_dev(wl.X, "bf16"), None, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    refp = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Yp), refp, False, f"cyclic proj q={q} M={M}")


def test_cyclic_plan_follows_M_and_stream_capture():
    """The cyclic schedule's tile sequences are planned on the host once per (handle, M).  One handle
    must give the explicit-types result for M1, then M2, then M1 again; and a first call with a new
    M inside stream capture (where the host cannot re-plan) must fall back to in-kernel planning."""
    q = 2
    cyc = binding.Proj([128] * q, [256] * q, dtype="bf16", schedule="cyclic")
    exp = binding.Proj([128] * q, [256] * q, dtype="bf16")
    W = H.to_dev(synth.normal(31, (128 * q, 256 * q), 0.05), "bf16")

    def pair(M, seed):
        X = H.to_dev(synth.normal(seed, (M, 128 * q), 1.0), "bf16")
        t = H.dev_types(synth.cyclic_types(M, q))
        return X, exp.forward(X, t, W, act="gelu")

    for M, seed in ((1024, 1), (2560, 2), (1024, 3), (770, 4)):
        X, want = pair(M, seed)
        assert torch.equal(cyc.forward(X, None, W, act="gelu"), want), M
    X, want = pair(1536, 5)                     # new M, first seen while capturing
    Y = torch.empty_like(want)
    ws = torch.empty(cyc.workspace_bytes(1536), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            cyc.forward(X, None, W, act="gelu", out=Y, workspace=ws, stream=stream)
    Y.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(Y, want) and cyc.last_status() == 0
    assert torch.equal(cyc.forward(X, None, W, act="gelu"), want)   # planned on the host now


def test_captured_graph_survives_later_calls_with_other_M():
    """A graph captured for M1 must not depend on the handle's plan cache: after eager calls with
    five other M (more than the cache holds) its replay still writes exactly the M1 result and
    nothing outside Y (canary rows behind it stay untouched)."""
    q = 2
    cyc = binding.Proj([128] * q, [256] * q, dtype="bf16", schedule="cyclic")
    exp = binding.Proj([128] * q, [256] * q, dtype="bf16")
    W = H.to_dev(synth.normal(33, (128 * q, 256 * q), 0.05), "bf16")
    M1 = 1024
    X1 = H.to_dev(synth.normal(34, (M1, 128 * q), 1.0), "bf16")
    want = exp.forward(X1, H.dev_types(synth.cyclic_types(M1, q)), W, act="gelu")
    assert torch.equal(cyc.forward(X1, None, W, act="gelu"), want)       # M1 is in the cache now
    buf = torch.full((M1 + 64, 256 * q), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(cyc.workspace_bytes(M1), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    stream.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            cyc.forward(X1, None, W, act="gelu", out=buf[:M1], workspace=ws, stream=stream)
    torch.cuda.current_stream().wait_stream(stream)
    for k, M2 in enumerate((2560, 512, 768, 3072, 1280)):
        X2 = H.to_dev(synth.normal(40 + k, (M2, 128 * q), 1.0), "bf16")
        w2 = exp.forward(X2, H.dev_types(synth.cyclic_types(M2, q)), W, act="gelu")
        assert torch.equal(cyc.forward(X2, None, W, act="gelu"), w2), M2
    buf.fill_(7.0)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(buf[:M1], want) and torch.all(buf[M1:] == 7.0)
    assert cyc.last_status() == 0


def test_pilot_tensor_square_law_and_interval_schedule():
    """The law and shape of the paper's pilot FFN projections: Q_2 (x) Q_2 (36 block products,
    9/16 of the dense MACs), D = 768 = 4 x 192, F = 1536 = 4 x 384, interval schedule."""
    wl = synth.pilot_ffn(integer=True)
    keep = oracle.support(4, "q2pow")
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", table="q2pow")
    assert proj.gemm_count() == 36
    counts = np.bincount(wl.types, minlength=4)
    assert proj.macs(counts.tolist()) * 16 == 9 * wl.M * wl.D * wl.F
    Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep))
    wl = synth.pilot_ffn()
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", table="q2pow")
    Yf = _run_ffn(wl, ffn, torch.float32)
    rows = _sample_rows(wl, 160, seed=3)
    ref = oracle.ffn(wl.X[rows], wl.types[rows], wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=keep)
    H.assert_bf16_close(H.to_np(Yf[torch.from_numpy(rows).cuda()]), ref, False, "pilot tensor-square FFN")
    # decode step of the same layer
    d = synth.pilot_ffn(M=8)
    d.types = synth.interval_types(8, 4, 768, start=190)      # positions 190..197 straddle a type boundary
    Yd = _run_ffn(d, ffn, torch.float32)
    refd = oracle.ffn(d.X, d.types, d.W_up, d.W_down, d.d_widths, d.f_widths, keep=keep)
    H.assert_bf16_close(H.to_np(Yd), refd, False, "pilot decode")


@pytest.mark.parametrize("q,P,periods,dw,fw,table", [
    (4, 768, 8, 192, 384, "q2pow"),     # the pilot's schedule floor((p mod 768) / 192): runs of 192 rows, eight sequences
    (2, 256, 5, 128, 256, "qq_unequal"),  # runs of 128 rows; unequal widths keep the handle on the table-driven kernel
    (4, 4096, 1, 128, 256, "q2pow"),    # one period: runs of 1024 rows (256-row tiles where the widths allow them)
])
def test_interval_schedule_with_period_reads_runs_in_place(q, P, periods, dw, fw, table):
    """INTERVAL schedule of a table-driven handle: type = (row mod P) / (P / q).  No bucketing, no gather (two
    launches per FFN); same bits as the explicit-types path on the same kernel, projection bit-exact on integers."""
    M = P * periods
    types = synth.interval_types(M, q, P)
    d_w, f_w = [dw] * q, [fw] * q
    law = "q2pow"
    if table == "qq_unequal":
        d_w, f_w, law = [dw, 2 * dw], [fw, 2 * fw], "qq"
    wl = synth.make_workload("itv", config=7, variant=q * 100 + periods, dtype="bf16", q=q, M=M, D=sum(d_w), F=sum(f_w),
                             types=types, integer=True, d_widths=d_w, f_widths=f_w)
    keep = oracle.support(q, law)
    proj = binding.Proj(d_w, f_w, dtype="bf16", table=law, schedule="interval")
    if periods > 1:
        proj.set_option("interval_period", P)
    launches = binding.launch_count()
    Y = proj.forward(H.to_dev(wl.X, "bf16"), None, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert proj.last_status() == 0 and binding.launch_count() - launches == 1
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, d_w, f_w, keep=keep))
    # the FFN on real data: interval schedule against explicit types on the same kernel, and against the oracle
    wr = synth.make_workload("itvr", config=7, variant=q * 100 + periods + 1, dtype="bf16", q=q, M=M, D=sum(d_w), F=sum(f_w),
                             types=types, d_widths=d_w, f_widths=f_w)
    f_int = binding.FFN(d_w, f_w, dtype="bf16", table=law, schedule="interval")
    if periods > 1:
        f_int.set_option("interval_period", P)
    f_exp = binding.FFN(d_w, f_w, dtype="bf16", table=law, schedule="explicit")
    f_exp.set_option("gemm_kernel", 1)
    launches = binding.launch_count()
    Y_int = _run_ffn(wr, f_int, torch.float32, types=False)
    assert binding.launch_count() - launches == 2
    Y_exp = _run_ffn(wr, f_exp, torch.float32)
    assert torch.equal(Y_int, Y_exp)
    rows = _sample_rows(wr, 64, seed=5)
    ref = oracle.ffn(wr.X[rows], wr.types[rows], wr.W_up, wr.W_down, d_w, f_w, keep=keep)
    H.assert_bf16_close(H.to_np(Y_int[torch.from_numpy(rows).cuda()]), ref, False, "interval FFN")
    # a batch that is no whole number of periods is refused
    with pytest.raises(binding.AlgError):
        proj.forward(H.to_dev(wl.X[:M - 64], "bf16"), None, H.to_dev(wl.W_up, "bf16"))


def _random_ffn_case(k):
    rng = np.random.default_rng(500 + k)
    q = int(rng.choice([1, 2, 3, 4, 8, 16, 32]))
    dw = int(rng.choice([8, 64, 128])) * int(rng.integers(1, 4))
    fw = int(rng.choice([8, 64, 128])) * int(rng.integers(1, 4))
    schedule = str(rng.choice(["cyclic", "explicit"]))
    M = int(rng.integers(1, 40)) * q if rng.random() < 0.5 else int(rng.integers(1, 3000))
    return q, M, dw, fw, schedule, int(rng.choice([0, 1, 4]))


@pytest.mark.parametrize("k", range(24))
def test_ffn_random_shapes_integer_bit_exact(k):
    """Seeded random group counts, widths on and off the tile grid, row counts, schedules and kernel choices; with
    act = none and entries in {-1, 0, 1} both projections are exact integer arithmetic."""
    q, M, dw, fw, schedule, kernel = _random_ffn_case(k)
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else synth.uniform_types(31 + k, M, q)
    wl = synth.make_workload("ffnfz", config=7, variant=700 + k, dtype="bf16", q=q, M=M, D=dw * q, F=fw * q, types=types,
                             integer=True)
    wl.X = np.sign(wl.X).astype(np.float32)
    wl.W_up = (np.sign(wl.W_up) * (np.abs(wl.W_up) > 2)).astype(np.float32)
    wl.W_down = np.sign(wl.W_down).astype(np.float32)
    Hh = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if np.abs(Hh).max() > 256:
        pytest.skip("hidden state not exactly representable in bf16")
    ffn = binding.FFN(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    try:
        ffn.set_option("gemm_kernel", kernel)
    except binding.AlgError:
        pass   # the handle's widths do not fit that kernel: the library's choice runs
    t = None if schedule == "cyclic" else H.dev_types(wl.types)
    Y = ffn.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), H.to_dev(wl.W_down, "bf16"), act=None,
                    out_dtype=torch.float32)
    assert ffn.last_status() == 0
    assert np.array_equal(H.to_np(Y), oracle.proj(Hh, wl.types, wl.W_down, wl.f_widths, wl.d_widths)), (q, M, dw, fw, schedule, kernel)
