"""GPU parity of the gated (SwiGLU) FFN, Y = (silu(X * W_gate) .* (X * W_up)) * W_down with the merged
gate/up bank, against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_32814_b200 import binding, synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run(wl, Wg, table="qq", schedule="explicit", out_dtype=torch.float32, kernel=None):
    ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16", table=table, schedule=schedule)
    if kernel is not None:
        ffn.set_option("gemm_kernel", kernel)
    Wgu = np.concatenate([Wg, wl.W_up], axis=1)          # the merged bank: [W_gate | W_up]
    Y = ffn.forward(H.to_dev(wl.X, "bf16"), None if schedule == "cyclic" else H.dev_types(wl.types),
                    H.to_dev(Wgu, "bf16"), H.to_dev(wl.W_down, "bf16"), out_dtype=out_dtype)
    assert ffn.last_status() == 0
    return Y, ffn


def _sample_rows(wl, per_type, seed=0):
    rng = np.random.default_rng(seed)
    rows = []
    for t in range(wl.q):
        idx = np.flatnonzero(wl.types == t)
        if idx.size:
            tail = idx[(idx.size // 128) * 128:]
            rows.append(np.concatenate([idx[:2], idx[-2:], tail[:2], rng.choice(idx, size=min(per_type, idx.size), replace=False)]))
    return np.unique(np.concatenate(rows))


@pytest.mark.parametrize("q,M,D,F,schedule", [
    (2, 700, 256, 512, "explicit"),      # ragged buckets, two hidden tiles per group
    (2, 1024, 128, 256, "cyclic"),       # type-strided A view
    (3, 515, 192, 384, "explicit"),      # non-power-of-two q, one hidden tile per group
    (1, 300, 128, 384, "explicit"),      # q = 1: an ordinary gated MLP
])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("kernel", [1, 4])   # the table-driven kernel, the large-algebra kernel
def test_gated_ffn_small_shapes(q, M, D, F, schedule, out_dtype, kernel):
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else synth.uniform_types(600 + q, M, q)
    wl, Wg = synth.gated_ffn("gated", q, M, D, F, types, variant=q * 10 + M % 7)
    # weights of the test are scaled up so that the hidden state is of order one
    wl.W_up, Wg, wl.W_down = (synth.bf16_round(w * 4.0) for w in (wl.W_up, Wg, wl.W_down))
    Y, ffn = _run(wl, Wg, schedule=schedule, out_dtype=out_dtype, kernel=kernel)
    ref = oracle.ffn_swiglu(wl.X, wl.types, Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"gated q={q} M={M}")
    counts = np.bincount(wl.types, minlength=q).tolist()
    keep = oracle.support(q)
    assert ffn.macs(counts) == 2 * oracle.macs(keep, wl.d_widths, wl.f_widths, counts) + \
        oracle.macs(keep, wl.f_widths, wl.d_widths, counts)


def test_gated_hidden_state_alone():
    """W_down = identity blocks turns the output into the hidden state of the row's own group:
    checks silu(gate) * up itself, on values spread over [-8, 8]."""
    q, M, D = 1, 256, 128
    F = 128
    X = synth.bf16_round(np.linspace(-8, 8, M * D, dtype=np.float32).reshape(M, D))
    Wg = np.eye(D, F, dtype=np.float32)
    Wu = synth.bf16_round(synth.normal(5, (D, F), 0.5))
    Wd = np.eye(F, D, dtype=np.float32)
    ffn = binding.GatedFFN([D], [F], dtype="bf16")
    t = torch.zeros(M, dtype=torch.int32, device="cuda")
    Y = ffn.forward(H.to_dev(X, "bf16"), t, H.to_dev(np.concatenate([Wg, Wu], axis=1), "bf16"), H.to_dev(Wd, "bf16"),
                    out_dtype=torch.float32)
    ref, Hh = oracle.ffn_swiglu(X, np.zeros(M, np.int32), Wg, Wu, Wd, [D], [F], return_hidden=True)
    got = H.to_np(Y)
    # Y is the bf16-rounded hidden state: half an ulp of bf16 plus the activation's own error
    assert np.all(np.abs(got - Hh) <= 2.0 ** -8 * np.abs(Hh) + 2e-3), float(np.abs(got - Hh).max())


def test_gated_pilot_shape_tensor_square_law():
    """The paper's pilot FFN: D = 768 = 4 x 192, F = 1536 = 4 x 384, bias-free SwiGLU under the
    tensor-square law Q_2 (x) Q_2, interval schedule."""
    M = 4 * 1536
    wl, Wg = synth.gated_ffn("pilot-gated", 4, M, 768, 1536, synth.interval_types(M, 4, 768), variant=1)
    keep = oracle.support(4, "q2pow")
    Y, ffn = _run(wl, Wg, table="q2pow")
    rows = _sample_rows(wl, 128, seed=4)
    ref = oracle.ffn_swiglu(wl.X[rows], wl.types[rows], Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=keep)
    got = H.to_np(Y[torch.from_numpy(rows).cuda()])
    assert H.rel_fro(got, ref) <= H.BF16_REL_FRO
    assert H.max_abs(got, ref) <= H.BF16_MAX_ABS
    counts = np.bincount(wl.types, minlength=4).tolist()
    assert ffn.macs(counts) * 16 == 9 * 3 * M * 768 * 1536          # (3/4)^2 of the dense 3 M D F


def test_gated_pilot_interval_schedule_in_place():
    """The pilot's typing floor((p mod 768) / 192) as the handle's schedule: the merged gate/up kernel reads the runs
    of a type in place and the down projection writes them back in place -- two launches, no types array, and the
    same bits as the explicit-types path on the same kernel."""
    M = 4 * 768
    types = synth.interval_types(M, 4, 768)
    wl, Wg = synth.gated_ffn("pilot-gated-itv", 4, M, 768, 1536, types, variant=3)
    Wgu = H.to_dev(np.concatenate([Wg, wl.W_up], axis=1), "bf16")
    Xd, Wd = H.to_dev(wl.X, "bf16"), H.to_dev(wl.W_down, "bf16")
    f_int = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16", table="q2pow", schedule="interval")
    f_int.set_option("interval_period", 768)
    launches = binding.launch_count()
    Y_int = f_int.forward(Xd, None, Wgu, Wd, out_dtype=torch.float32)
    assert f_int.last_status() == 0 and binding.launch_count() - launches == 2
    f_exp = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16", table="q2pow")
    f_exp.set_option("gemm_kernel", 1)
    Y_exp = f_exp.forward(Xd, H.dev_types(types), Wgu, Wd, out_dtype=torch.float32)
    assert torch.equal(Y_int, Y_exp)
    rows = _sample_rows(wl, 48, seed=6)
    keep = oracle.support(4, "q2pow")
    ref = oracle.ffn_swiglu(wl.X[rows], wl.types[rows], Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths, keep=keep)
    H.assert_bf16_close(H.to_np(Y_int[torch.from_numpy(rows).cuda()]), ref, False, "gated interval")
    # options the run view does not have
    with pytest.raises(binding.AlgError):
        f_int.set_option("stage_k", 32)
    with pytest.raises(binding.AlgError):
        f_int.set_option("interval_period", 4 * 96)        # runs of 96 rows: no multiple of 64
    with pytest.raises(binding.AlgError):
        f_exp.set_option("interval_period", 768)           # not an interval handle


def test_gated_kernel_table_shape_q32():
    """One shape of the paper's gated-FFN table: 4096 -> 12288 -> 4096 at q = 32 (group widths 128
    and 384), M = 2048 rows, i.i.d. row types."""
    q, M, D, F = 32, 2048, 4096, 12288
    wl, Wg = synth.gated_ffn("gated-q32", q, M, D, F, synth.uniform_types(632, M, q), variant=2)
    Y, ffn = _run(wl, Wg)
    rows = np.unique(np.concatenate([np.arange(0, M, 16), [M - 1]]))
    ref = oracle.ffn_swiglu(wl.X[rows], wl.types[rows], Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    got = H.to_np(Y[torch.from_numpy(rows).cuda()])
    assert H.rel_fro(got, ref) <= H.BF16_REL_FRO
    assert H.max_abs(got, ref) <= H.BF16_MAX_ABS


@pytest.mark.parametrize("q,M,dw,fw", [
    (32, 300, 64, 192),      # 2048 -> 6144 at q = 32: hidden groups of 192 columns, two 96-column tiles each
    (32, 257, 80, 304),      # 2560 -> 9728: groups of 80 and 304 (reductions of 80 and 304 are no multiples of 64)
    (32, 2048, 64, 24),      # 2048 -> 768 (an expert): hidden groups of 24 columns; cyclic: two types per tile
    (32, 32 * 200, 64, 192), # cyclic: 200 rows per type, two m-tiles each
    (32, 333, 224, 64),      # 7168 -> 2048 (an expert)
    (4, 1000, 64, 192),      # the same group widths at small q: several m-tiles per type
    (3, 515, 80, 304),
    (1, 1, 64, 24),          # one row
])
@pytest.mark.parametrize("schedule", ["explicit", "cyclic"])
def test_gated_ffn_groups_off_the_tile_grid(q, M, dw, fw, schedule):
    """Gated FFN whose groups are no multiples of 128 columns (the public model shapes of the paper's gated-FFN table
    split 32 ways): both projections on the large-algebra kernel, hidden state in bucketed order."""
    types = synth.cyclic_types(M, q) if schedule == "cyclic" else synth.uniform_types(700 + q + M, M, q)
    wl, Wg = synth.gated_ffn("gated-off-grid", q, M, q * dw, q * fw, types, variant=q + dw + fw)
    wl.W_up, Wg, wl.W_down = (synth.bf16_round(w * 2.0) for w in (wl.W_up, Wg, wl.W_down))
    n0 = binding.launch_count()
    Y, ffn = _run(wl, Wg, schedule=schedule, out_dtype=torch.bfloat16)
    if schedule == "cyclic" and M % q == 0 and M > 1:
        assert binding.launch_count() - n0 == 2      # equal buckets: rows read and written in place, no bucketing, no gather
    rows = np.unique(np.concatenate([_sample_rows(wl, 6, seed=3), np.arange(min(M, 8))])) if M > 64 else np.arange(M)
    ref = oracle.ffn_swiglu(wl.X[rows], wl.types[rows], Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y[torch.from_numpy(rows).cuda()]), ref, True, f"gated off-grid q={q} M={M}")


@pytest.mark.parametrize("q,dw,fw", [
    (32, 64, 192),       # 2048 -> 6144
    (32, 80, 304),       # 2560 -> 9728
    (32, 128, 384),      # 4096 -> 12288
    (32, 64, 24),        # 2048 -> 768
    (32, 224, 64),       # 7168 -> 2048
    (2, 128, 256),       # few wide groups: strips narrower than a group
    (5, 40, 72),
])
@pytest.mark.parametrize("M", [1, 3, 8])
def test_gated_decode_step_in_one_launch(q, dw, fw, M):
    """Decode rows of the gated FFN against the oracle.  One row is one launch (two matrix-vector phases around a
    bounded wait; twice in a row on the same handle: the counters are cleared by the kernel); a few rows go through
    the prefill kernels.  Types explicit and cyclic."""
    for schedule in ("explicit", "cyclic"):
        types = synth.cyclic_types(M, q) if schedule == "cyclic" else synth.uniform_types(800 + q + M, M, q)
        wl, Wg = synth.gated_ffn("gated-decode", q, M, q * dw, q * fw, types, variant=q + dw + M)
        wl.W_up, Wg, wl.W_down = (synth.bf16_round(w * 2.0) for w in (wl.W_up, Wg, wl.W_down))
        ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16", schedule=schedule)
        Wgu, Wd, X = H.to_dev(np.concatenate([Wg, wl.W_up], axis=1), "bf16"), H.to_dev(wl.W_down, "bf16"), H.to_dev(wl.X, "bf16")
        t = None if schedule == "cyclic" else H.dev_types(types)
        ref = oracle.ffn_swiglu(wl.X, wl.types, Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
        for out_dtype in (torch.float32, torch.bfloat16):
            n0 = binding.launch_count()
            Y = ffn.forward(X, t, Wgu, Wd, out_dtype=out_dtype)
            assert ffn.last_status() == 0 and (M > 1 or binding.launch_count() - n0 == 1)
            H.assert_bf16_close(H.to_np(Y), ref, out_dtype == torch.bfloat16, f"gated decode q={q} M={M} {schedule}")
        # the prefill kernels on the same rows agree within the tolerance of two bf16 paths
        ffn.set_option("small_m_kernel", 0)
        Y2 = ffn.forward(X, t, Wgu, Wd, out_dtype=torch.float32)
        H.assert_bf16_close(H.to_np(Y2), ref, False, "prefill kernels on decode rows")


def test_gated_decode_row_type_out_of_range_gives_a_zero_row():
    q, dw, fw = 4, 64, 128
    wl, Wg = synth.gated_ffn("gated-decode-bad", q, 1, q * dw, q * fw, np.array([0], np.int32), variant=9)
    ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16")
    Wgu, Wd, X = H.to_dev(np.concatenate([Wg, wl.W_up], axis=1), "bf16"), H.to_dev(wl.W_down, "bf16"), H.to_dev(wl.X, "bf16")
    for out_dtype in (torch.float32, torch.bfloat16):
        Y = torch.full((1, q * dw), 3.0, dtype=out_dtype, device="cuda")
        ffn.forward(X, H.dev_types(np.array([7], np.int32)), Wgu, Wd, out=Y)
        assert ffn.last_status() == 5
        assert np.all(H.to_np(Y) == 0)
    # the handle is usable afterwards
    Y = ffn.forward(X, H.dev_types(np.array([2], np.int32)), Wgu, Wd, out_dtype=torch.float32)
    ref = oracle.ffn_swiglu(wl.X, np.array([2], np.int32), Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(Y), ref, False, "after a bad type")


def test_gated_decode_bounded_wait_expires_and_the_handle_recovers():
    """The wait between the two phases of the one-launch decode step is bounded: made to expect an arrival that never
    comes (nothing faults, every CTA leaves), it gives up after the limit, the status says so, and the next calls on
    the same handle are right again."""
    q, dw, fw = 32, 64, 192
    wl, Wg = synth.gated_ffn("gated-decode-wait", q, 1, q * dw, q * fw, np.array([9], np.int32), variant=4)
    ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16")
    args = (H.to_dev(wl.X, "bf16"), H.dev_types(wl.types), H.to_dev(np.concatenate([Wg, wl.W_up], axis=1), "bf16"),
            H.to_dev(wl.W_down, "bf16"))
    ref = oracle.ffn_swiglu(wl.X, wl.types, Wg, wl.W_up, wl.W_down, wl.d_widths, wl.f_widths)
    H.assert_bf16_close(H.to_np(ffn.forward(*args, out_dtype=torch.float32)), ref, False, "before")
    ffn.set_option("wait_limit_cycles", 6_000_000)       # about 3 ms
    ffn.set_option("test_stall_bytes", 512)
    ffn.forward(*args, out_dtype=torch.float32)
    assert ffn.last_status() == 6
    ffn.set_option("test_stall_bytes", 0)
    ffn.set_option("wait_limit_cycles", 4_000_000_000)
    for _ in range(2):
        H.assert_bf16_close(H.to_np(ffn.forward(*args, out_dtype=torch.float32)), ref, False, "after")
    assert ffn.last_status() == 0


def test_gated_refusals():
    with pytest.raises(binding.AlgError) as e:
        binding.GatedFFN([64, 128], [192, 320], dtype="bf16")     # hidden groups off the 128-column grid and unequal
    assert e.value.code == 2
    with pytest.raises(binding.AlgError):
        binding.GatedFFN([64, 64], [128, 128], dtype="f32")


@pytest.mark.parametrize("M", [1, 3])
def test_gated_decode_chain_in_a_graph_replays(M):
    """Five dependent gated layers (distinct weights, layer l+1 reads layer l's output) captured in one CUDA graph, as
    the benchmark's decode chain does: consecutive launches overlap through programmatic dependent launch (every launch
    requests its weights before the one before it has finished) and share the handle's exchange counters.  Every replay
    reproduces, bit for bit, the layers run one at a time with a device synchronisation between them; that result is
    checked against the oracle layer by layer."""
    q, dw, fw, L = 32, 64, 192, 5
    types = synth.uniform_types(77, M, q)
    wl, _ = synth.gated_ffn("gated-chain", q, M, q * dw, q * fw, types, variant=1)
    D, F = q * dw, q * fw
    ffn = binding.GatedFFN(wl.d_widths, wl.f_widths, dtype="bf16")
    ffn.set_option("small_m_kernel", 3)
    t = H.dev_types(types)
    # (weights large enough that the activations do not die out along the chain: the gated map is quadratic in x)
    Wgu_h = [synth.bf16_round(synth.normal(300 + l, (D, 2 * F), 0.12)) for l in range(L)]
    Wd_h = [synth.bf16_round(synth.normal(400 + l, (F, D), 0.12)) for l in range(L)]
    Wgu, Wd = [H.to_dev(w, "bf16") for w in Wgu_h], [H.to_dev(w, "bf16") for w in Wd_h]
    acts = [H.to_dev(wl.X, "bf16")] + [torch.zeros((M, D), dtype=torch.bfloat16, device="cuda") for _ in range(L)]
    ws = torch.empty(ffn.workspace_bytes(M), dtype=torch.uint8, device="cuda")
    want = [acts[0]]
    for l in range(L):       # one layer at a time
        n0 = binding.launch_count()
        want.append(ffn.forward(want[l], t, Wgu[l], Wd[l], workspace=ws))
        assert binding.launch_count() - n0 == 1
        torch.cuda.synchronize()
        ref = oracle.ffn_swiglu(H.to_np(want[l]), types, Wgu_h[l][:, :F], Wgu_h[l][:, F:], Wd_h[l], wl.d_widths, wl.f_widths)
        assert H.rel_fro(H.to_np(want[l + 1]), ref) <= H.BF16_REL_FRO, f"layer {l}"    # (magnitudes grow along the chain)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        for l in range(L):   # back to back, overlapping
            ffn.forward(acts[l], t, Wgu[l], Wd[l], out=acts[l + 1], workspace=ws, stream=stream)
        stream.synchronize()
        for l in range(L):
            assert torch.equal(acts[l + 1], want[l + 1]), f"eager layer {l}"
        with torch.cuda.graph(g, stream=stream):
            for l in range(L):
                ffn.forward(acts[l], t, Wgu[l], Wd[l], out=acts[l + 1], workspace=ws, stream=stream)
    for rep in range(4):
        for l in range(L):
            acts[l + 1].zero_()
        g.replay()
        torch.cuda.synchronize()
        for l in range(L):
            assert torch.equal(acts[l + 1], want[l + 1]), f"replay {rep} layer {l}"
    assert ffn.last_status() == 0
