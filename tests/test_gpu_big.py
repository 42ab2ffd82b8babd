"""GPU parity of the large-algebra path (q up to 256, equal group widths in multiples of 8 that need not
fit the GPU tile; Section "Kernel Benchmarks", appendix "Large Projections and Square Products") against
the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _types(schedule, M, q, seed):
    if schedule == "cyclic":
        return synth.cyclic_types(M, q)
    if schedule == "interval":
        return (np.arange(M) // (M // q)).astype(np.int32)
    return synth.uniform_types(1000 + seed, M, q)


def _workload(q, M, s_w, r_w, schedule, integer=True, seed=1):
    return synth.make_workload("big", config=9, variant=seed, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q,
                               types=_types(schedule, M, q, seed), integer=integer, with_down=False)


def _forward(wl, schedule, out_dtype, **kw):
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    assert proj.kernel_path(wl.M) == binding.ALG_PATH_TCGEN05
    t = H.dev_types(wl.types) if schedule == "explicit" else None
    Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype, **kw)
    assert proj.last_status() == 0
    return Y, proj


@pytest.mark.parametrize("q,M,s_w,r_w,schedule", [
    (64, 64 * 48, 32, 64, "cyclic"),        # q > 32; 48 rows per type: every tile is ragged
    (40, 40 * 130, 24, 40, "interval"),     # widths no multiple of 16: zero-padded stage, 8-column store masks; 128 + 2 rows
    (256, 256 * 8, 8, 16, "cyclic"),        # the largest algebra, the narrowest groups
    (128, 128 * 16, 40, 200, "interval"),   # 5120 -> 25600 at q = 128: blocks of 40 x 200
    (48, 48 * 256, 64, 128, "interval"),    # 64-deep stages, two full m-tiles per type
    (8, 1000, 160, 800, "explicit"),        # q <= 32 with widths off the tile grid: bucketing + gather, four 208-wide tiles
    (4, 515, 80, 304, "explicit"),          # two 160-wide column tiles per group, the second one 144 wide
    (2, 300, 72, 136, "cyclic"),            # equal buckets of 150 rows, 136 = 128 + 8 columns
    (3, 301, 24, 40, "cyclic"),             # q does not divide M: counted buckets
    (5, 640, 96, 264, "explicit"),          # two column tiles of 144 and 120
    (64, 3000, 32, 64, "explicit"),         # q > 32 with i.i.d. types: bucketing tables for 256 types, ragged buckets
    (256, 4000, 8, 16, "explicit"),         # some types get a handful of rows
    (40, 1003, 24, 40, "cyclic"),           # q > 32 and q does not divide M
    (256, 256 * 16, 20, 100, "interval"),   # widths that are multiples of 4 only: the q = 256 split of 5120 -> 25600
    (64, 64 * 130, 20, 100, "cyclic"),      # the same blocks, two m-tiles per type, type-strided rows
    (12, 777, 100, 36, "explicit"),         # groups deeper than one stage (64 + 36): full and zero-padded stages share the ring
    (4, 300, 132, 292, "explicit"),         # three stages per group, two column tiles (160 + 132)
    (48, 48 * 8, 4, 4, "interval"),         # the narrowest groups there are
    (35, 35 * 40, 24, 40, "cyclic"),        # three types per tile, the last tile holds two; type-strided rows
    (35, 35 * 40, 24, 40, "interval"),
    (50, 50, 16, 24, "interval"),           # one row per type: fifty types in one tile
    (7, 7 * 64, 64, 128, "interval"),       # two types per tile, the last one alone
    (20, 20 * 33, 8, 264, "cyclic"),        # 33 rows per type (three per tile, boxes off the 8-row swizzle atom), two column tiles
    # several narrow output groups per tile (taken when at least four tiles per SM remain):
    (40, 40 * 150, 72, 40, "cyclic"),       # five groups per tile (200 columns); 128 + 22 rows per type
    (48, 4800, 136, 104, "explicit"),       # two groups per tile, the second one across three 64-column boxes; counted buckets
    (64, 64 * 130, 24, 24, "interval"),     # ten groups per tile, the last tile four; groups straddle the 64-column boxes
    (32, 32 * 200, 100, 88, "cyclic"),      # widths of 4 only in the reduction (repacked), two groups per tile
    # several types AND several groups per tile (panel segments of the types first, then one diagonal segment per group;
    # groups that share a unit with the tile's own types come one by one):
    (256, 256 * 8, 100, 20, "interval"),    # 25600 -> 5120 at q = 256, M = 2048: sixteen types x seven groups, repacked
    (128, 128 * 16, 200, 40, "cyclic"),     # eight types x three groups, cyclic rows
    (200, 200 * 8, 24, 24, "interval"),     # a last type group of eight types, a last unit of fewer groups
    (160, 160 * 40, 16, 104, "interval"),   # three types of 40 rows x two groups of 104 columns (three boxes)
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_big_integer_bit_exact(q, M, s_w, r_w, schedule, out_dtype):
    wl = _workload(q, M, s_w, r_w, schedule, seed=q + M % 13)
    Y, proj = _forward(wl, schedule, out_dtype)
    assert proj.gemm_count() == 2 * q * q - q
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"{len(bad)} mismatches, first at {bad[:5].tolist()}"


@pytest.mark.parametrize("q,M,s_w,r_w,schedule", [
    (64, 64 * 48, 32, 64, "cyclic"),
    (40, 40 * 130, 24, 40, "interval"),
    (4, 515, 80, 304, "explicit"),
])
def test_big_stage_depth_32_same_bits(q, M, s_w, r_w, schedule):
    """32-deep stages (64-byte rows of X, 64-byte swizzle atoms) are the other pipeline for the same sums."""
    wl = _workload(q, M, s_w, r_w, schedule, seed=q + 3)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    proj.set_option("stage_k", 32)
    t = H.dev_types(wl.types) if schedule == "explicit" else None
    Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=torch.float32)
    assert proj.last_status() == 0
    assert np.array_equal(H.to_np(Y), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))


def _random_case(k):
    rng = np.random.default_rng(4242 + k)
    q = int(rng.choice([1, 2, 3, 5, 7, 12, 24, 33, 47, 64, 96, 130, 200, 256]))
    s_w = 8 * int(rng.integers(1, 13 if q < 100 else 5))
    r_w = 8 * int(rng.integers(1, 41 if q < 40 else (13 if q < 100 else 5)))
    schedule = str(rng.choice(["cyclic", "interval", "explicit"]))
    rows = int(rng.integers(1, 300 if q < 40 else 40))
    M = q * rows if schedule == "interval" or rng.random() < 0.5 else int(rng.integers(1, q * rows + 1))
    return q, M, s_w, r_w, schedule


@pytest.mark.parametrize("k", range(24))
def test_big_random_shapes_integer_bit_exact(k):
    """Seeded random algebra sizes, block shapes, row counts and schedules (whichever kernel the library picks)."""
    q, M, s_w, r_w, schedule = _random_case(k)
    wl = _workload(q, M, s_w, r_w, schedule, seed=100 + k)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    t = H.dev_types(wl.types) if schedule == "explicit" else None
    out_dtype = torch.float32 if k % 2 else torch.bfloat16
    Y = proj.forward(H.to_dev(wl.X, "bf16"), t, H.to_dev(wl.W_up, "bf16"), out_dtype=out_dtype)
    assert proj.last_status() == 0
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    bad = np.argwhere(H.to_np(Y) != ref)
    assert bad.size == 0, f"case {(q, M, s_w, r_w, schedule)}: {len(bad)} mismatches, first at {bad[:5].tolist()}"


def test_big_is_the_square_product_of_two_algebra_elements():
    """Eqs. q-product-diag / q-product-off: C = A * B for n x n arrays of b x b blocks equals the typed
    projection of A's rows (block row i has type i) through B."""
    n, b = 1024, 64
    q = n // b
    wl = _workload(q, n, b, b, "interval", seed=5)
    Y, proj = _forward(wl, "interval", torch.float32)
    ref = oracle.square(wl.X, wl.W_up, [b] * q, [b] * q, [b] * q)
    assert np.array_equal(H.to_np(Y), ref)
    rows = [n // q] * q
    assert proj.macs(rows) == oracle.macs(oracle.support(q), [b] * q, [b] * q, rows)


def test_big_counts_follow_the_law_at_large_q():
    q = 96
    proj = binding.Proj([16] * q, [24] * q, dtype="bf16", schedule="cyclic")
    keep = oracle.support(q)
    rows = list(range(1, q + 1))
    assert proj.gemm_count() == oracle.gemm_count(keep) == 2 * q * q - q
    assert proj.macs(rows) == oracle.macs(keep, [16] * q, [24] * q, rows)


def test_big_bias_gelu_normal_data_and_strides():
    q, M, s_w, r_w = 64, 64 * 40, 40, 104
    wl = _workload(q, M, s_w, r_w, "cyclic", integer=False, seed=3)
    bias = synth.bf16_round(synth.normal(77, (q * r_w,), 0.1))
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="cyclic")
    # operands and result inside wider allocations
    Xp = torch.zeros(M, q * s_w + 24, dtype=torch.bfloat16, device="cuda")
    Xp[:, :q * s_w] = H.to_dev(wl.X, "bf16")
    Wp = torch.zeros(q * s_w, q * r_w + 8, dtype=torch.bfloat16, device="cuda")
    Wp[:, :q * r_w] = H.to_dev(wl.W_up, "bf16")
    out = torch.full((M, q * r_w + 16), 7.0, dtype=torch.float32, device="cuda")
    proj.forward(Xp[:, :q * s_w], None, Wp[:, :q * r_w], bias=H.to_dev(bias, "bf16"), act="gelu", out=out[:, :q * r_w])
    assert proj.last_status() == 0
    ref = oracle.gelu_array(oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths, bias=bias))
    got = out[:, :q * r_w].cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 5e-3
    assert np.abs(got - ref).max() <= 2e-2
    assert torch.all(out[:, q * r_w:] == 7.0)      # nothing is written past N


@pytest.mark.parametrize("q,M,s_w,r_w", [(4, 600, 40, 72), (48, 700, 16, 24)])
def test_big_static_scratch_and_bad_type(q, M, s_w, r_w):
    wl = _workload(q, M, s_w, r_w, "explicit", seed=11)
    types = wl.types.copy()
    types[17] = q + 3
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="explicit")
    out = torch.empty(M, q * r_w, dtype=torch.float32, device="cuda")
    proj.forward_static(H.to_dev(wl.X, "bf16"), H.dev_types(types), H.to_dev(wl.W_up, "bf16"), out)
    assert proj.last_status() == 5
    good = np.arange(M) != 17
    ref = oracle.proj(wl.X[good], wl.types[good], wl.W_up, wl.d_widths, wl.f_widths)
    got = out.cpu().numpy()
    assert np.array_equal(got[good], ref)
    assert not got[17].any()


def test_big_forward_host_matches_device_call():
    q, M, s_w, r_w = 64, 64 * 20, 24, 56
    wl = _workload(q, M, s_w, r_w, "interval", seed=21)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="interval")
    W = H.to_dev(wl.W_up, "bf16")
    Xh = torch.from_numpy(wl.X.astype(np.float32)).to(torch.bfloat16).pin_memory()
    Yh = torch.empty(M, q * r_w, dtype=torch.float32).pin_memory()
    proj.forward_host(Xh, None, W, Yh)
    torch.cuda.synchronize()
    assert proj.last_status() == 0
    assert np.array_equal(Yh.numpy(), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))


def test_big_refusals():
    with pytest.raises(binding.AlgError):      # unequal widths at q > 32
        binding.Proj([32] * 63 + [64], [64] * 64, dtype="bf16", schedule="cyclic")
    with pytest.raises(binding.AlgError):      # widths that are no multiple of 4
        binding.Proj([18] * 64, [100] * 64, dtype="bf16", schedule="cyclic")
    with pytest.raises(binding.AlgError):
        binding.Proj([32] * 64, [64] * 64, dtype="f32", schedule="cyclic")
    with pytest.raises(binding.AlgError):
        binding.Proj([32] * 64, [64] * 64, dtype="bf16", table="dense", schedule="cyclic")
    with pytest.raises(binding.AlgError):
        binding.Proj([8] * 257, [8] * 257, dtype="bf16", schedule="cyclic")
    proj = binding.Proj([32] * 64, [64] * 64, dtype="bf16", schedule="interval")
    X = torch.zeros(100, 64 * 32, dtype=torch.bfloat16, device="cuda")
    W = torch.zeros(64 * 32, 64 * 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.AlgError):      # q must divide M
        proj.forward(X, None, W)
    with pytest.raises(binding.AlgError):
        proj.set_option("gemm_kernel", 2)


def test_weights_packed_once():
    """Group widths that are multiples of 4 only: the bank padded once by alg_proj_pack_weight gives the same bits as the
    per-call padding, with one launch fewer per call; handles that pad nothing have nothing to pack."""
    q, M, s_w, r_w = 256, 256 * 8, 100, 20
    wl = _workload(q, M, s_w, r_w, "interval", seed=77)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule="interval")
    X, W = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16")
    n0 = binding.launch_count()
    Y0 = proj.forward(X, None, W, out_dtype=torch.float32)
    per_call = binding.launch_count() - n0
    assert proj.packed_weight_bytes() == (q * 104) * (q * 24) * 2
    Wp = proj.pack_weight(W)
    proj.set_option("weight_packed", 1)
    n0 = binding.launch_count()
    Y1 = proj.forward(X, None, Wp, out_dtype=torch.float32)
    assert binding.launch_count() - n0 == per_call - 1 and proj.last_status() == 0
    assert torch.equal(Y0, Y1)
    assert np.array_equal(H.to_np(Y1), oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths))
    plain = binding.Proj([64] * 40, [128] * 40, dtype="bf16", schedule="interval")
    assert plain.packed_weight_bytes() == 0
    with pytest.raises(binding.AlgError):
        plain.set_option("weight_packed", 1)
    with pytest.raises(binding.AlgError):
        plain.pack_weight(torch.zeros((64 * 40, 128 * 40), dtype=torch.bfloat16, device="cuda"))


@pytest.mark.parametrize("k", range(16))
def test_big_many_small_types_and_narrow_groups_random(k):
    """Random shapes in the regime where a tile takes several types and several groups: many types of few rows, groups of
    at most 112 columns, widths in multiples of 4 (padded per call or packed once); integers exact."""
    rng = np.random.default_rng(31000 + k)
    q = int(rng.choice([64, 96, 128, 160, 200, 256]))
    rows = int(rng.choice([1, 2, 3, 5, 8, 12, 16, 24, 33, 40, 64]))
    s_w, r_w = 4 * int(rng.integers(1, 17)), 4 * int(rng.integers(1, 29))
    if (q * s_w) % 8 or (q * r_w) % 8:
        s_w, r_w = 2 * s_w, 2 * r_w
    schedule = str(rng.choice(["cyclic", "interval"]))
    wl = _workload(q, q * rows, s_w, r_w, schedule, seed=700 + k)
    proj = binding.Proj(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
    W = H.to_dev(wl.W_up, "bf16")
    if proj.packed_weight_bytes() and k % 2 == 0:
        W = proj.pack_weight(W)
        proj.set_option("weight_packed", 1)
    out_dtype = torch.float32 if k % 2 else torch.bfloat16
    Y = proj.forward(H.to_dev(wl.X, "bf16"), None, W, out_dtype=out_dtype)
    assert proj.last_status() == 0
    ref = oracle.proj(wl.X, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    if out_dtype == torch.bfloat16:
        ref = H.bf16_rne(ref)
    assert np.array_equal(H.to_np(Y), ref), (q, rows, s_w, r_w, schedule)
