"""GPU parity of the two gradient maps of the projection (dX, dW) against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _problem(q, M, s_w, r_w, types=None, integer=True, seed=1):
    if types is None:
        types = synth.uniform_types(5000 + seed, M, q)
    wl = synth.make_workload("grad", config=8, variant=500 + seed, dtype="bf16", q=q, M=M, D=s_w * q, F=r_w * q, types=types,
                             integer=integer, with_down=False)
    G = synth.small_ints(synth.seed_for(8, 900 + seed), (M, r_w * q)) if integer else \
        synth.bf16_round(synth.normal(synth.seed_for(8, 900 + seed), (M, r_w * q), 1.0))
    return wl, G


@pytest.mark.parametrize("q,M,s_w,r_w,schedule", [
    (2, 300, 128, 128, "explicit"),     # one tile per block, ragged buckets
    (2, 1000, 384, 256, "explicit"),    # several tiles, both endpoint products
    (3, 515, 128, 256, "explicit"),     # non-power-of-two q
    (4, 777, 128, 512, "explicit"),     # config-3 group shapes
    (1, 200, 256, 256, "explicit"),     # q = 1: the gradients of an ordinary GEMM
    (2, 1024, 256, 128, "cyclic"),      # cyclic schedule, whole 64-row blocks per type: X and G read in place
    (4, 4 * 192, 128, 384, "cyclic"),   # in place, three reduction blocks per type, four segments on the diagonal
    (3, 3 * 64, 384, 128, "cyclic"),    # in place, one block per type, several feature tiles
    (2, 1000, 128, 256, "cyclic"),      # 500 rows per type: not whole blocks, padded copies
])
def test_grad_maps_integer_bit_exact(q, M, s_w, r_w, schedule):
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else None
    wl, G = _problem(q, M, s_w, r_w, types=types, seed=q * 7 + M % 5)
    g = binding.ProjGrad(wl.d_widths, wl.f_widths, schedule=schedule)
    t = None if schedule == "cyclic" else H.dev_types(wl.types)
    Xd, Wd, Gd = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16"), H.to_dev(G, "bf16")
    dX = g.grad_input(Gd, t, Wd, out_dtype=torch.float32)
    dW = g.grad_weight(Xd, Gd, t)
    assert g.last_status() == 0
    ref_dx = oracle.proj_vjp_x(G, wl.types, wl.W_up, wl.d_widths, wl.f_widths)
    ref_dw = oracle.proj_vjp_w(wl.X, G, wl.types, wl.d_widths, wl.f_widths)
    bad = np.argwhere(H.to_np(dX) != ref_dx)
    assert bad.size == 0, f"dX: {len(bad)} mismatches, first {bad[:5].tolist()}"
    bad = np.argwhere(H.to_np(dW) != ref_dw)
    assert bad.size == 0, f"dW: {len(bad)} mismatches, first {bad[:5].tolist()}"
    # repeatable bit for bit (one owner per output element, no atomics)
    assert torch.equal(dW, g.grad_weight(Xd, Gd, t)) and torch.equal(dX, g.grad_input(Gd, t, Wd, out_dtype=torch.float32))


def test_grad_tables_missing_type_and_bad_type():
    q, M, s_w, r_w = 4, 600, 128, 128
    wl, G = _problem(q, M, s_w, r_w, seed=9)
    Xd, Wd, Gd = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16"), H.to_dev(G, "bf16")
    for table in ("dense", "q2pow"):
        keep = oracle.support(q, table)
        g = binding.ProjGrad(wl.d_widths, wl.f_widths, table=table)
        assert np.array_equal(H.to_np(g.grad_input(Gd, H.dev_types(wl.types), Wd, out_dtype=torch.float32)),
                              oracle.proj_vjp_x(G, wl.types, wl.W_up, wl.d_widths, wl.f_widths, keep=keep)), table
        assert np.array_equal(H.to_np(g.grad_weight(Xd, Gd, H.dev_types(wl.types))),
                              oracle.proj_vjp_w(wl.X, G, wl.types, wl.d_widths, wl.f_widths, keep=keep)), table
    # a type with no rows: its private weight blocks get a zero gradient
    types = np.where(wl.types == 3, 1, wl.types).astype(np.int32)
    g = binding.ProjGrad(wl.d_widths, wl.f_widths)
    dW = H.to_np(g.grad_weight(Xd, Gd, H.dev_types(types)))
    assert np.array_equal(dW, oracle.proj_vjp_w(wl.X, G, types, wl.d_widths, wl.f_widths))
    assert not dW[3 * s_w:, :3 * r_w].any()
    # an out-of-range type: status raised, the row contributes to no block and gets a zero input gradient
    types[5] = 11
    dW = H.to_np(g.grad_weight(Xd, Gd, H.dev_types(types)))
    assert g.last_status() == 5
    good = np.ones(M, bool)
    good[5] = False
    assert np.array_equal(dW, oracle.proj_vjp_w(wl.X[good], G[good], types[good], wl.d_widths, wl.f_widths))
    dX = H.to_np(g.grad_input(Gd, H.dev_types(types), Wd, out_dtype=torch.float32))
    assert g.last_status() == 5 and not dX[5].any()
    assert np.array_equal(dX[good], oracle.proj_vjp_x(G[good], types[good], wl.W_up, wl.d_widths, wl.f_widths))


def test_grad_config2_up_projection_normal_data():
    """The up projection of configuration 2 (768 -> 3072, M = 8192, type = position mod 2), real-valued
    data: both gradients within the bf16 tolerance of the fp64 oracle (dW on a sample of its rows)."""
    wl = synth.config2()
    G = synth.bf16_round(synth.normal(synth.seed_for(2, 77), (wl.M, wl.F), 1.0))
    g = binding.ProjGrad(wl.d_widths, wl.f_widths, schedule="cyclic")
    Xd, Wd, Gd = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_up, "bf16"), H.to_dev(G, "bf16")
    dX = g.grad_input(Gd, None, Wd, out_dtype=torch.float32)
    dW = g.grad_weight(Xd, Gd, None)
    rows = np.arange(0, wl.M, 16)
    ref_dx = oracle.proj_vjp_x(G[rows], wl.types[rows], wl.W_up, wl.d_widths, wl.f_widths)
    got = H.to_np(dX[torch.from_numpy(rows).cuda()])
    assert H.rel_fro(got, ref_dx) <= H.BF16_REL_FRO and H.max_abs(got, ref_dx) <= H.BF16_MAX_ABS
    ref_dw = oracle.proj_vjp_w(wl.X, G, wl.types, wl.d_widths, wl.f_widths)
    got = H.to_np(dW)
    assert H.rel_fro(got, ref_dw) <= 1e-4        # exact bf16 products, fp32 accumulation over 4096-8192 rows
    assert np.abs(got - ref_dw).max() <= 2e-2 + 1e-4 * np.abs(ref_dw).max()


def test_grad_refusals():
    with pytest.raises(binding.AlgError) as e:
        binding.ProjGrad([64, 64], [72, 72])      # output groups the tensor-core tiles do not divide
    assert e.value.code == 2
