"""GPU parity of alg_proj_forward against the CPU oracle (single projections)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run_proj(wl, *, table="qq", custom=None, bias=None, act=None, out_dtype=None, which="up", schedule="explicit",
              expect_path=None, kernel=None):
    s, r = (wl.d_widths, wl.f_widths) if which == "up" else (wl.f_widths, wl.d_widths)
    W = wl.W_up if which == "up" else wl.W_down
    proj = binding.Proj(s, r, dtype=wl.dtype, table=table, custom_keep=custom, schedule=schedule)
    if kernel is not None:
        proj.set_option("gemm_kernel", kernel)
    if expect_path is not None:
        assert proj.kernel_path(wl.M) == expect_path
    X = H.to_dev(wl.X, wl.dtype)
    Wd = H.to_dev(W, wl.dtype)
    bd = None if bias is None else H.to_dev(bias, wl.dtype)
    Y = proj.forward(X, H.dev_types(wl.types), Wd, bias=bd, act=act, out_dtype=out_dtype)
    assert proj.last_status() == 0
    return Y, proj


# ---- config 1: fp32, true fp32 FMAs ---------------------------------------------------------

def test_cfg1_integer_bit_exact():
    wl = synth.config1(integer=True)
    Y, proj = _run_proj(wl, expect_path=binding.ALG_PATH_SIMT)
    assert proj.gemm_count() == 6
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    got = Y.cpu().numpy()
    assert got.dtype == np.float32
    assert np.array_equal(got.view(np.uint32), ref.astype(np.float32).view(np.uint32))


def test_cfg1_normal_fp32():
    wl = synth.config1()
    Y, _ = _run_proj(wl)
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    got = H.to_np(Y)
    assert H.rel_fro(got, ref) <= H.F32_REL_FRO
    assert H.max_abs(got, ref) <= H.F32_MAX_ABS


def test_cfg1_dense_table_is_matmul():
    wl = synth.config1(integer=True)
    Y, proj = _run_proj(wl, table="dense")
    assert proj.gemm_count() == 8
    assert np.array_equal(H.to_np(Y), wl.X.astype(np.float64) @ wl.W_up.astype(np.float64))


# ---- SIMT path on awkward shapes (any q, unequal widths, ragged everything) ------------------

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_simt_ragged_unequal_widths(dtype):
    q, s, r, M = 3, [24, 40, 8], [72, 8, 136], 333
    rng_types = synth.uniform_types(7, M, q)
    wl = synth.make_workload("ragged", config=9, variant=1, dtype=dtype, q=q, M=M, D=sum(s), F=sum(r),
                             types=rng_types, integer=True, with_down=False, d_widths=s, f_widths=r)
    bias = synth.small_ints(99, (sum(r),))
    Y, proj = _run_proj(wl, bias=bias, out_dtype=torch.float32, expect_path=binding.ALG_PATH_SIMT)
    assert proj.gemm_count() == 15
    ref = oracle.proj(wl.X, wl.types, wl.W_up, s, r, bias=bias)
    assert np.array_equal(H.to_np(Y), ref)


# ---- tensor-core path: integer data is exact in bf16 x bf16 -> fp32 -------------------------

def _tc_workload(q, M, s_w, r_w, types=None, integer=True, seed=1):
    if types is None:
        types = synth.uniform_types(1000 + seed, M, q)
    return synth.make_workload("tc", config=8, variant=seed, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q,
                               types=types, integer=integer, with_down=False)


@pytest.mark.parametrize("q,M,s_w,r_w", [
    (2, 128, 64, 128),     # one tile per pair, one or two k-blocks
    (2, 300, 128, 256),    # ragged last m-tile, 256-wide tiles
    (2, 1000, 384, 384),   # 128-wide tiles (384 = 3 x 128), six k-blocks per group
    (4, 777, 128, 512),    # config-3 group shapes, several types
    (3, 515, 192, 128),    # non-power-of-two q
    (1, 200, 256, 256),    # q = 1 degenerates to an ordinary GEMM
    (2, 700, 1024, 192),   # long K loops (32 K blocks per off-diagonal tile), 192 columns wide
    (2, 300, 1024, 256),
    (1, 520, 1024, 128),
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("kernel", [0, 1, 4])   # the library's choice, the table-driven kernel, the large-algebra kernel
def test_tc_integer_bit_exact(q, M, s_w, r_w, out_dtype, kernel):
    wl = _tc_workload(q, M, s_w, r_w, seed=q * 10 + M % 7)
    Y, proj = _run_proj(wl, out_dtype=out_dtype, expect_path=binding.ALG_PATH_TCGEN05, kernel=kernel)
    assert proj.gemm_count() == 2 * q * q - q
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    got = H.to_np(Y)
    bad = np.argwhere(got != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"


# ---- CTA-pair kernel (tcgen05 cta_group::2), selected through a handle option --------------------

@pytest.mark.parametrize("q,M,s_w,r_w,schedule", [
    (1, 700, 512, 384, "explicit"),    # 256-wide tile plus the 128-wide remainder tile, ragged last 256-row tile
    (2, 300, 128, 256, "explicit"),    # short K loops, one full tile per group
    (2, 1337, 256, 384, "explicit"),   # several m-tiles per type, remainder tiles, both endpoint products
    (3, 515, 64, 128, "explicit"),     # only 128-wide tiles, single K block per group
    (2, 1026, 128, 384, "cyclic"),     # type-strided A view, arithmetic row scatter
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_pair_kernel_integer_bit_exact(q, M, s_w, r_w, schedule, out_dtype):
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else None
    wl = _tc_workload(q, M, s_w, r_w, types=types, seed=q * 31 + M % 11)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    proj.set_option("gemm_kernel", 2)
    launches = binding.launch_count()
    Y = proj.forward(H.to_dev(wl.X, "bf16"), None if schedule == "cyclic" else H.dev_types(wl.types),
                     H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype)
    assert proj.last_status() == 0
    assert binding.launch_count() - launches == (1 if schedule == "cyclic" else 3)   # bucketing, gather, GEMM
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"
    # the one-CTA kernel on the same handle gives the same bits
    proj.set_option("gemm_kernel", 1)
    Y1 = proj.forward(H.to_dev(wl.X, "bf16"), None if schedule == "cyclic" else H.dev_types(wl.types),
                      H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype)
    assert torch.equal(Y, Y1)


# ---- one-CTA kernel with 256-row tiles (two accumulators per tile) -------------------------------

@pytest.mark.parametrize("q,M,s_w,r_w,schedule", [
    (1, 700, 512, 384, "explicit"),    # ragged last 256-row tile, three column tiles
    (2, 300, 128, 128, "explicit"),    # buckets smaller than one tile
    (2, 1337, 256, 384, "explicit"),   # several tiles per type, both endpoint products
    (3, 515, 64, 128, "explicit"),
    (2, 1026, 128, 384, "cyclic"),     # type-strided A view with 256-row boxes, arithmetic row scatter
    (4, 4096, 64, 128, "cyclic"),      # 1024 rows per type: the library picks this tiling by itself
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_tall_tiles_integer_bit_exact(q, M, s_w, r_w, schedule, out_dtype):
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else None
    wl = _tc_workload(q, M, s_w, r_w, types=types, seed=q * 37 + M % 13)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    if M < 4096:
        proj.set_option("gemm_kernel", 3)
    t = None if schedule == "cyclic" else H.dev_types(wl.types)
    Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype)
    assert proj.last_status() == 0
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"
    proj.set_option("gemm_kernel", 1)      # 128-row tiles on the same handle: same bits
    assert torch.equal(Y, proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype))


def test_tall_tiles_bias_gelu_normal_data():
    wl = _tc_workload(2, 2500, 384, 384, integer=False, seed=19)
    bias = synth.bf16_round(synth.normal(21, (wl.F,), 0.5))
    for act, out_dtype in (("gelu", torch.float32), ("gelu", torch.bfloat16), (None, torch.bfloat16)):
        proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")   # 1250 rows per type: 256-row tiles by default
        Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"),
                         bias=H.to_dev(bias, "bf16"), act=act, out_dtype=out_dtype)
        assert proj.last_status() == 0
        ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, bias=bias)
        if act:
            ref = oracle.gelu_array(ref)
        H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"256-row tiles act={act}")


def test_pair_kernel_bias_gelu_normal_data_and_refusal():
    wl = _tc_workload(2, 900, 384, 384, integer=False, seed=13)
    bias = synth.bf16_round(synth.normal(15, (wl.F,), 0.5))
    for act, out_dtype in (("gelu", torch.float32), ("gelu", torch.bfloat16), (None, torch.bfloat16)):
        proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
        proj.set_option("gemm_kernel", 2)
        Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(wl.W_up, "bf16"),
                         bias=H.to_dev(bias, "bf16"), act=act, out_dtype=out_dtype)
        assert proj.last_status() == 0
        ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, bias=bias)
        if act:
            ref = oracle.gelu_array(ref)
        H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"pair kernel act={act}")
    # a shape the pair kernel cannot tile (192-wide groups) refuses the option and keeps working
    odd = binding.Proj([64, 64], [192, 192], dtype="bf16")
    with pytest.raises(binding.AlgError) as e:
        odd.set_option("gemm_kernel", 2)
    assert e.value.code == 2
    with pytest.raises(binding.AlgError):
        odd.set_option("tile_n", 256)
    wl2 = _tc_workload(2, 260, 64, 192, seed=17)
    Y = odd.forward(H.to_dev(wl2.X, "bf16"), H.dev_types(wl2.types), H.to_dev(wl2.W_up, "bf16"), out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), oracle.proj(wl2.X, wl2.types, wl2.W_up, wl2.d_widths, wl2.f_widths))


def test_bucketing_beyond_65536_rows():
    """More rows than the one-kernel bucketing covers: the per-chunk histogram + scatter pair of
    kernels builds the permutation (ragged everything: M is odd, the types are i.i.d.)."""
    wl = _tc_workload(4, 70001, 64, 128, seed=23)
    Y, proj = _run_proj(wl, out_dtype=torch.float32, expect_path=binding.ALG_PATH_TCGEN05)
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"
    types = wl.types.copy()
    types[[5, 66000, 70000]] = [4, -3, 99]           # out-of-range types in the first and the last chunk
    Yb = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(types), H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert proj.last_status() == 5
    got = H.to_np(Yb)
    assert not got[[5, 66000, 70000]].any()
    good = np.ones(wl.M, bool)
    good[[5, 66000, 70000]] = False
    assert np.array_equal(got[good], ref[good])


@pytest.mark.parametrize("M", [1, 1023, 1025, 2048, 2049, 4097, 8191, 8192, 8193, 16384, 16385])
def test_bucketing_across_the_cluster_sizes(M):
    """Up to 8192 rows (16384 where the device takes clusters of 16) the bucketing kernel is one cluster of
    1 ... 16 CTAs that exchange their counts through shared memory; one row more takes the variant with the
    counter in global memory.  Skewed types
    (one type absent, one holding half the rows), bit-exact on integer data, and an out-of-range type in the
    last row."""
    q = 4
    wl = _tc_workload(q, M, 64, 128, seed=300 + M % 97)
    rng = np.random.default_rng(M)
    types = rng.choice(np.array([0, 2, 2, 3], np.int32), size=M)      # type 1 never occurs
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    Y = proj.forward(X, H.dev_types(types), W, out_dtype=torch.float32)
    assert proj.last_status() == 0
    ref = oracle.proj(wl.X, types, wl.W_up, wl.d_widths, wl.f_widths)
    assert np.array_equal(H.to_np(Y), ref)
    types[M - 1] = q + 5
    Yb = H.to_np(proj.forward(X, H.dev_types(types), W, out_dtype=torch.float32))
    assert proj.last_status() == 5
    assert not Yb[M - 1].any() and np.array_equal(Yb[:M - 1], ref[:M - 1])


def test_options_tile_width_and_in_kernel_plan():
    """Every tile width that divides the groups, and both ways of planning the cyclic schedule,
    give the same bits."""
    M, q = 1024, 2
    wl = _tc_workload(q, M, 128, 768, types=synth.cyclic_types(M, q), seed=29)
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    for tile_n in (0, 128, 192, 256):
        proj.set_option("tile_n", tile_n)
        for host_plan in (1, 0):
            proj.set_option("host_plan", host_plan)
            Y = proj.forward(X, None, W, out_dtype=torch.float32)
            assert np.array_equal(H.to_np(Y), ref), (tile_n, host_plan)
    proj.set_option("small_m_kernel", 0)
    assert proj.kernel_path(8) == binding.ALG_PATH_TCGEN05
    Y8 = proj.forward(X[:8], None, W, out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y8), ref[:8])


@pytest.mark.parametrize("q,M,s_w,r_w,schedule,tile_n,kernel", [
    (2, 1000, 384, 768, "explicit", 256, 1),   # 8 stages of 24 KB, ragged tiles, both endpoint products
    (2, 1000, 384, 768, "explicit", 192, 1),
    (2, 1026, 128, 384, "cyclic", 128, 1),     # twelve stages of 16 KB, type-strided A view
    (2, 1337, 256, 384, "explicit", 0, 3),     # 256-row tiles: two A halves per stage
    (3, 515, 64, 128, "explicit", 0, 1),       # two K blocks of 32 per group
    (2, 2048, 1536, 384, "cyclic", 0, 3),      # long reduction through the ring many times over
])
def test_stage_depth_option_same_bits(q, M, s_w, r_w, schedule, tile_n, kernel):
    """Stages of 32 and of 64 reduction steps (64- and 128-byte swizzle atoms of the K-major operand) are two
    pipelines for the same arithmetic."""
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else None
    wl = _tc_workload(q, M, s_w, r_w, types=types, seed=q * 41 + M % 17)
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    proj.set_option("gemm_kernel", kernel)
    if tile_n:
        proj.set_option("tile_n", tile_n)
    t = None if schedule == "cyclic" else H.dev_types(wl.types)
    for stage_k in (32, 64, 0):
        proj.set_option("stage_k", stage_k)
        for host_plan in (1, 0):
            proj.set_option("host_plan", host_plan)
            Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
            assert proj.last_status() == 0
            bad = np.argwhere(H.to_np(Y) != ref)
            assert bad.size == 0, f"stage_k {stage_k}: {len(bad)} mismatches, first at {bad[:5].tolist()}"
    with pytest.raises(binding.AlgError):
        proj.set_option("stage_k", 48)


def test_tc_missing_type_and_single_row():
    wl = _tc_workload(2, 1, 128, 128, types=np.array([1], dtype=np.int32))
    Y, _ = _run_proj(wl, out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))
    wl = _tc_workload(4, 260, 64, 128, types=np.full(260, 2, dtype=np.int32))
    Y, _ = _run_proj(wl, out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))


def test_tc_dense_and_custom_tables():
    wl = _tc_workload(4, 400, 64, 128, seed=5)
    Y, proj = _run_proj(wl, table="dense", out_dtype=torch.float32)
    assert proj.gemm_count() == 64
    assert np.array_equal(H.to_np(Y), wl.X.astype(np.float64) @ wl.W_up.astype(np.float64))
    keep = oracle.support(4, "q2pow")  # the tensor-square law: 36 products
    Y, proj = _run_proj(wl, table="custom", custom=torch.from_numpy(keep), out_dtype=torch.float32)
    assert proj.gemm_count() == 36
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep))


@pytest.mark.parametrize("kernel", [1, 4])   # the table-driven kernel, the large-algebra kernel
def test_tc_bias_and_gelu_normal_data(kernel):
    wl = _tc_workload(2, 700, 384, 256, integer=False, seed=3)
    bias = synth.bf16_round(synth.normal(5, (wl.F,), 0.5))
    for act, out_dtype in (("gelu", torch.float32), ("gelu", torch.bfloat16), (None, torch.float32)):
        Y, _ = _run_proj(wl, bias=bias, act=act, out_dtype=out_dtype, kernel=kernel)
        ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, bias=bias)
        if act:
            ref = np.vectorize(oracle.gelu)(ref)
        H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"act={act}")


def test_cyclic_schedule_needs_no_types():
    wl = _tc_workload(2, 513, 128, 128, types=synth.cyclic_types(513, 2))
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    Y = proj.forward(H.to_dev(wl.X, "bf16"), None, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))


def test_strided_operands_and_determinism():
    wl = _tc_workload(2, 640, 128, 256, seed=11, integer=False)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    Xp = torch.zeros((wl.M, wl.D + 64), dtype=torch.bfloat16, device="cuda")
    Xp[:, :wl.D] = H.to_dev(wl.X, "bf16")
    Wp = torch.zeros((wl.D, wl.F + 8), dtype=torch.bfloat16, device="cuda")
    Wp[:, :wl.F] = H.to_dev(wl.W_up, "bf16")
    out = torch.full((wl.M, wl.F + 8), 7.0, dtype=torch.float32, device="cuda")
    t = H.dev_types(wl.types)
    proj.forward(Xp[:, :wl.D], t, Wp[:, :wl.F], out=out[:, :wl.F])
    first = out.clone()
    proj.forward(Xp[:, :wl.D], t, Wp[:, :wl.F], out=out[:, :wl.F])
    assert torch.equal(first, out)                       # run-to-run bitwise identical
    assert torch.all(out[:, wl.F:] == 7.0)               # padding columns untouched
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(out[:, :wl.F]), ref, False, "strided")


def test_bad_type_sets_status_and_zeroes_row():
    wl = _tc_workload(2, 300, 64, 128, seed=2)
    types = wl.types.copy()
    types[17] = 5
    types[200] = -1
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
    Y = proj.forward(H.to_dev(wl.X, "bf16"), H.dev_types(types), H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert proj.last_status() == 5          # ALG_ERR_BAD_TYPE
    assert proj.last_status() == 0          # reading clears it
    got = H.to_np(Y)
    assert not got[17].any() and not got[200].any()
    good = np.ones(300, bool)
    good[[17, 200]] = False
    ref = oracle.proj(wl.X[good], types[good], wl.W_up, wl.d_widths, wl.f_widths)
    assert np.array_equal(got[good], ref)


def test_argument_errors():
    proj = binding.Proj([128, 128], [128, 128], dtype="bf16")
    X = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((256, 256), dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(4, dtype=torch.int32, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.AlgError) as e:
        proj.forward(X, t, W, workspace=small)
    assert e.value.code == 3
    with pytest.raises(binding.AlgError) as e:
        proj.forward(X, None, W)            # explicit schedule without types
    assert e.value.code == 1
    Y = proj.forward(X[:0], t[:0], W)        # M = 0 is a no-op
    assert Y.shape == (0, 256)
    assert proj.macs([3, 5]) == 8 * (2 * 128 * 128) + 3 * 128 * 128 + 5 * 128 * 128


def test_gelu_epilogue_accuracy_on_a_dense_grid():
    """Identity weights turn the projection into a pure epilogue test: Y = gelu(x) in fp32.
    The kernel's branch-free erf-GELU must match the closed form to fp32 rounding level."""
    n = 128
    vals = np.concatenate([np.linspace(-9, 9, 128 * n - 64), [0.0] * 8, [-6.0, 6.0, -40.0, 40.0], np.zeros(52)])
    X = synth.bf16_round(vals.astype(np.float32).reshape(128, n))
    proj = binding.Proj([n], [n], dtype="bf16")
    W = torch.eye(n, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(128, dtype=torch.int32, device="cuda")
    Y = proj.forward(H.to_dev(X, "bf16"), t, W, act="gelu", out_dtype=torch.float32)
    ref = np.vectorize(oracle.gelu)(X.astype(np.float64))
    err = np.abs(H.to_np(Y) - ref)
    assert err.max() <= 4e-7 + 2e-7 * np.abs(ref).max(), err.max()
    Yt = proj.forward(H.to_dev(X, "bf16"), t, W, act="gelu_tanh", out_dtype=torch.float32)
    assert np.abs(H.to_np(Yt) - ref).max() <= 2e-3      # the tanh form is a different function


@pytest.mark.parametrize("q,M,dw,fw,kernel", [
    (2, 128, 128, 128, 1),       # one tile
    (4, 5000, 128, 512, 1),      # short reductions: the library's own choice is the in-kernel gather
    (3, 777, 256, 384, 1),       # ragged buckets, 192-column tiles
    (2, 4096, 384, 1536, 1),     # reductions of 384 and 768 columns
    (2, 8192, 384, 384, 3),      # 256-row tiles: two gathers per lane and stage
])
def test_row_gather_in_the_kernel_matches_the_copy_pass(q, M, dw, fw, kernel):
    """Explicit types, option ROW_GATHER: rows fetched through the permutation by the GEMM's producer warps (four rows
    per copy instruction) against the bucketed copy -- same bits, one launch fewer, integers exact against the oracle."""
    types = synth.uniform_types(900 + q, M, q)
    wl = synth.make_workload("rowg", config=7, variant=q * 10 + kernel, dtype="bf16", q=q, M=M, D=q * dw, F=q * fw,
                             types=types, integer=True, d_widths=[dw] * q, f_widths=[fw] * q)
    X, W, t = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16"), H.dev_types(types)
    out, launches = [], []
    for mode in (1, 2):
        proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16")
        proj.set_option("gemm_kernel", kernel)
        proj.set_option("row_gather", mode)
        n0 = binding.launch_count()
        out.append(proj.forward(X, t, W, out_dtype=torch.float32))
        launches.append(binding.launch_count() - n0)
        assert proj.last_status() == 0
    assert torch.equal(out[0], out[1])
    assert launches[0] == launches[1] + 1
    assert np.array_equal(H.to_np(out[1]), oracle.proj(wl.X, types, wl.W_up, wl.d_widths, wl.f_widths))
