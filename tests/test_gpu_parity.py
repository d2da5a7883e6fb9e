"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  Small problems are compared element by element over every output;
the 720p-class, 1080p and sweep workloads are compared on sampled queries and key rows
plus whole-tensor invariants (see parity_util).  Tolerances are stated in parity_util."""
import math

import pytest
import torch

import parity_util as pu
from paper_2607_22696_b200 import binding, inputs

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32


def small_problem(T, H, W, heads, d, window, dtype, sigma, seed):
    wl = inputs.Workload("case", T, H, W, heads, d, tuple(window), dtype, sigma, seed)
    t = inputs.make_inputs(wl, "cpu", with_dout=True)
    return t["q"], t["k"], t["v"], t["offsets"], t["dout"]


def test_extension_is_loaded():
    lib = binding.load()
    assert lib.dsa3d_status_string(0) == b"success"


# ----------------------------------------------------------------- BASELINE configs 1, 2

def test_config_tiny_f32_forward_backward():
    wl = inputs.WORKLOADS["tiny_f32"]
    t = inputs.make_inputs(wl, "cpu")
    pu.full_parity(t["q"], t["k"], t["v"], t["offsets"], t["dout"], wl.window)


def test_config_480p_bf16_forward_full():
    wl = inputs.WORKLOADS["480p_bf16_fwd"]
    t = inputs.make_inputs(wl, "cuda")
    q, k, v, off = (t[n].cpu() for n in ("q", "k", "v", "offsets"))
    pu.full_parity(q, k, v, off, None, wl.window, check_backward=False)


# ------------------------------------------------------------- small cases, every output

@pytest.mark.parametrize("dtype", [F32, BF16])
@pytest.mark.parametrize("d", [32, 64, 128])
def test_head_dims_and_ragged_item_counts(dtype, d):
    # 5*7*9*3 = 945 items: not a multiple of any block's group count
    pu.full_parity(*small_problem(5, 7, 9, 3, d, (3, 3, 3), dtype, 1.0, 20 + d), (3, 3, 3))


@pytest.mark.parametrize("window", [(1, 1, 1), (2, 2, 2), (3, 5, 5), (3, 7, 7), (4, 8, 8)])
def test_windows(window):
    sigma = 1.5
    pu.full_parity(*small_problem(4, 9, 10, 2, 64, window, BF16, sigma, 31), window)
    pu.full_parity(*small_problem(3, 6, 7, 2, 32, window, F32, sigma, 32), window)


@pytest.mark.parametrize("dims", [(1, 9, 11), (6, 1, 11), (6, 9, 1), (1, 1, 1), (1, 1, 40)])
def test_grid_dimensions_of_one(dims):
    pu.full_parity(*small_problem(*dims, 2, 32, (3, 3, 3), F32, 0.7, 33), (3, 3, 3))
    pu.full_parity(*small_problem(*dims, 2, 128, (3, 3, 3), BF16, 0.7, 34), (3, 3, 3))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_zero_and_integer_offsets(dtype):
    q, k, v, off, dout = small_problem(5, 6, 7, 2, 64, (3, 3, 3), dtype, 1.0, 35)
    pu.full_parity(q, k, v, torch.zeros_like(off), dout, (3, 3, 3))
    ioff = inputs.uniform_int(off.shape, 36, 3, -3, 3, torch.float32)      # reaches -1 and size exactly
    pu.full_parity(q, k, v, ioff, dout, (3, 3, 3))


@pytest.mark.parametrize("dtype", [F32, BF16])
def test_out_of_range_nan_and_huge_offsets(dtype):
    q, k, v, off, dout = small_problem(4, 5, 6, 2, 32, (3, 3, 3), dtype, 1.0, 37)
    far = torch.full_like(off, 100.0)
    pu.full_parity(q, k, v, far, dout, (3, 3, 3))                        # every sample dead
    mixed = off.clone()
    flat = mixed.view(-1, 3)
    flat[0::7, 0] = float("nan")
    flat[1::7, 1] = float("inf")
    flat[2::7, 2] = -float("inf")
    flat[3::7, 0] = 3e38
    flat[4::7, 1] = -1e30
    pu.full_parity(q, k, v, mixed, dout, (3, 3, 3))


def test_positions_near_cell_boundaries_take_the_fp32_decision():
    """Offsets a hair away from integers: the cell is decided by the fp32 position, the
    same way on both sides, so even dOffsets agrees."""
    q, k, v, off, dout = small_problem(3, 40, 60, 1, 32, (3, 3, 3), F32, 1.0, 38)
    near = torch.round(off) + (inputs.normal(off.shape, 39, 3, 1.0, torch.float32) * 1e-6)
    pu.full_parity(q, k, v, near, dout, (3, 3, 3))


def test_per_query_outputs_are_run_to_run_deterministic():
    q, k, v, off, dout = (z.cuda() for z in small_problem(6, 10, 12, 4, 128, (3, 3, 3), BF16, 1.5, 40))
    dims = tuple(q.shape)
    o1, l1 = pu.gpu_forward(q, k, v, off, dims, (3, 3, 3))
    g1 = pu.gpu_backward(q, k, v, off, l1, dout, dims, (3, 3, 3))
    o2, l2 = pu.gpu_forward(q, k, v, off, dims, (3, 3, 3))
    g2 = pu.gpu_backward(q, k, v, off, l2, dout, dims, (3, 3, 3))
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
    assert torch.equal(g1[0], g2[0]) and torch.equal(g1[3], g2[3])
    for a, b in ((g1[1], g2[1]), (g1[2], g2[2])):        # atomics: order may differ
        assert float((a.float() - b.float()).abs().max()) <= 2e-2 * float(a.float().abs().max())


def test_binding_reports_library_errors():
    z = torch.zeros(4 * 8 * 8 * 2 * 48, device="cuda")
    off = torch.zeros(4 * 8 * 8 * 2 * 27 * 3, device="cuda")
    lse = torch.zeros(4 * 8 * 8 * 2, device="cuda")
    with pytest.raises(binding.Dsa3dError) as e:
        binding.dsa3d_forward(z, z, z, off, 4, 8, 8, 2, 48, (3, 3, 3), z, lse)
    assert e.value.status == 3


# ------------------------------------------------- BASELINE configs 3, 4, 5 at full size

def _tile_route(t, dims, window, fixed_window):
    """The pair of entry points `bench.py` times for workloads with zero offsets (fixed-window pair) or
    offsets below 1 in size (bounded-offsets pair)."""
    T, H, W, heads, d = dims
    out, lse = torch.full_like(t["q"], float("nan")), torch.full((T, H, W, heads), float("nan"), device="cuda")
    grads = [torch.full_like(t["q"], float("nan")) for _ in range(3)] + [torch.full_like(t["offsets"], float("nan"))]
    sizes = binding.dsa3d_backward_fixed_window_workspace_bytes if fixed_window else binding.dsa3d_backward_bounded_offsets_workspace_bytes
    ws = torch.full((max(sizes(T, H, W, heads, d, window, t["q"].dtype), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    if fixed_window:
        binding.dsa3d_forward_fixed_window(t["q"], t["k"], t["v"], T, H, W, heads, d, window, out, lse)
        binding.dsa3d_backward_fixed_window(t["q"], t["k"], t["v"], lse, t["dout"], T, H, W, heads, d, window, *grads, ws)
    else:
        binding.dsa3d_forward_bounded_offsets(t["q"], t["k"], t["v"], t["offsets"], T, H, W, heads, d, window, out, lse)
        binding.dsa3d_backward_bounded_offsets(t["q"], t["k"], t["v"], t["offsets"], lse, t["dout"], T, H, W, heads, d,
                                               window, *grads, ws)
    torch.cuda.synchronize()
    assert binding.dsa3d_device_timeout_flag() == 0
    return out, lse, tuple(grads)


def run_large(name, heads_sel, key_boxes, n_random=1024, backward=True, route="general"):
    wl = inputs.WORKLOADS[name]
    dims = (wl.T, wl.H, wl.W, wl.heads, wl.d)
    t = inputs.make_inputs(wl, "cuda", with_dout=True) if route != "general" else inputs.make_inputs(wl, "cuda")
    grads = None
    if route != "general":
        out, lse, grads = _tile_route(t, dims, wl.window, route == "fixed_window")
        t["out"] = out
        pu.assert_bilinearity_invariants(t, out, grads)
    else:
        out, lse = pu.gpu_forward(t["q"], t["k"], t["v"], t["offsets"], dims, wl.window)
        t["out"] = out
    if backward and route == "general":
        grads = pu.gpu_backward(t["q"], t["k"], t["v"], t["offsets"], lse, t["dout"], dims, wl.window)
        pu.assert_bilinearity_invariants(t, out, grads)
    pu.sampled_parity(t, dims, wl.window, lse, grads, heads_sel, n_random=n_random, key_boxes=key_boxes)
    del t, out, lse, grads
    torch.cuda.empty_cache()


def test_config_720p_bf16_forward_backward():
    run_large("720p_bf16", [0, 11, 23], [((0, 0, 0), (2, 2, 2)), ((31, 22, 40), (32, 24, 42)),
                                          ((63, 44, 78), (64, 45, 80))])


def test_config_720p_bf16_every_element():
    """The whole 720p-class workload (708 M elements per tensor) against a full oracle run
    (about a minute on 16 host cores): every element of every output inside the bound."""
    wl = inputs.WORKLOADS["720p_bf16"]
    dims = (wl.T, wl.H, wl.W, wl.heads, wl.d)
    t = inputs.make_inputs(wl, "cuda")
    out, lse = pu.gpu_forward(t["q"], t["k"], t["v"], t["offsets"], dims, wl.window)
    grads = pu.gpu_backward(t["q"], t["k"], t["v"], t["offsets"], lse, t["dout"], dims, wl.window)
    host = {n: z.cpu() for n, z in t.items()}
    del t
    torch.cuda.empty_cache()
    import oracle
    o_ref, l_ref = oracle.forward(host["q"], host["k"], host["v"], host["offsets"], *dims, wl.window)
    pu.assert_close("out", out, o_ref, wl.dtype)
    pu.assert_close("lse", lse, l_ref, wl.dtype)
    del o_ref, l_ref, out, lse
    refs = oracle.backward(host["q"], host["k"], host["v"], host["offsets"], host["dout"], *dims, wl.window)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), grads, refs):
        pu.assert_close(name, got, ref, wl.dtype, backward=True)


def test_config_1080p_256f_bf16_forward_backward():
    run_large("1080p_256f_bf16", [0, 7, 15], [((0, 0, 0), (2, 2, 2)), ((128, 33, 60), (129, 35, 62)),
                                               ((255, 67, 118), (256, 68, 120))])


def test_paper_window_3x7x7_on_the_1080p_grid():
    run_large("1080p_64f_w377_bf16", [0, 15], [((0, 0, 0), (1, 1, 2)), ((32, 33, 60), (33, 34, 61))], n_random=256)


@pytest.mark.parametrize("kind", ["zero", "int", "normal"])
@pytest.mark.parametrize("window", ["222", "333", "355"])
def test_config_sweep_720p_grid(window, kind):
    boxes = [((0, 0, 0), (1, 2, 2)), ((32, 22, 40), (33, 23, 42))]
    run_large(f"sweep_w{window}_{kind}", [0, 15], boxes, n_random=512)


@pytest.mark.parametrize("name,route", [("sweep_w222_zero", "fixed_window"), ("sweep_w333_zero", "fixed_window"),
                                        ("sweep_w355_zero", "fixed_window"), ("sweep_w377_zero", "fixed_window"),
                                        ("sweep_w333_small", "bounded")])
def test_sweep_grid_through_the_entry_points_the_bench_times(name, route):
    """Zero offsets and offsets below 1 in size at the sweep's full grid, through the entry points
    `bench.py` uses for them (tensor-core tile kernels): sampled queries and key boxes against the oracle,
    whole-tensor invariants."""
    boxes = [((0, 0, 0), (1, 2, 2)), ((32, 22, 40), (33, 23, 42)), ((63, 44, 78), (64, 45, 80))]
    run_large(name, [0, 15], boxes, n_random=512, route=route)


# ------------------------------------------------- tilings of the backward dK/dV scatter

@pytest.mark.parametrize("tiling", ["0", "2,2,2,1", "4,8,8,0", "1,1,1,3", "3,5,7,2", "4,8,8,6"])
def test_backward_is_the_same_for_every_tiling(tiling, monkeypatch):
    """dK/dV are pre-reduced per query tile for corners inside the tile's halo and sent
    straight to the accumulators otherwise; any split of the work (none tiled, tiles that
    do not divide the grid, no halo, one-query tiles) must give the oracle's result."""
    monkeypatch.setenv("DSA3D_TILE", tiling)
    q, k, v, off, dout = small_problem(5, 11, 13, 3, 128, (3, 3, 3), BF16, 1.7, 50)
    pu.full_parity(q, k, v, off, dout, (3, 3, 3))
    q, k, v, off, dout = small_problem(3, 9, 10, 2, 64, (2, 2, 2), BF16, 0.8, 51)
    pu.full_parity(q, k, v, off, dout, (2, 2, 2))


def test_large_window_through_the_tile_kernel():
    pu.full_parity(*small_problem(4, 10, 12, 2, 128, (3, 7, 7), BF16, 2.0, 52), (3, 7, 7))


# ------------------------------------------------------------- host-buffer entry point

@pytest.mark.parametrize("dtype,shape", [(BF16, (6, 10, 12, 3, 64)), (F32, (6, 10, 12, 3, 64)),
                                         (BF16, (19, 9, 10, 2, 128)), (F32, (11, 5, 6, 2, 32)),
                                         (BF16, (1, 7, 9, 2, 64))])
def test_step_host_matches_the_device_entry_points(dtype, shape):
    """dsa3d_step_host (pinned host buffers in, pinned host buffers out, the step pipelined
    over slabs of frames with the copies on side streams) must return what dsa3d_forward +
    dsa3d_backward return on device buffers; run twice to catch a stale event or buffer.
    The shapes give two slabs, several slabs with a ragged last one (on tile boundaries for
    bf16, two frames each for fp32), and a single frame."""
    q, k, v, off, dout = small_problem(*shape, (3, 3, 3), dtype, 1.3, 60)
    dims = tuple(q.shape)
    dev = [z.cuda() for z in (q, k, v, off, dout)]
    out_d, lse_d = pu.gpu_forward(*dev[:4], dims, (3, 3, 3))
    g_d = pu.gpu_backward(*dev[:4], lse_d, dev[4], dims, (3, 3, 3))
    pin = lambda z: z.clone().pin_memory()
    hin = [pin(z) for z in (q, k, v, off, dout)]
    hout = {n: torch.full_like(q, float("nan")).pin_memory() for n in ("out", "dq", "dk", "dv")}
    hout["lse"] = torch.full(dims[:4], float("nan")).pin_memory()
    hout["doff"] = torch.full_like(off, float("nan")).pin_memory()
    arena = torch.empty(binding.dsa3d_step_host_arena_bytes(*dims, (3, 3, 3), dtype), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        binding.dsa3d_step_host(*hin, *dims, (3, 3, 3), hout["out"], hout["lse"], hout["dq"], hout["dk"],
                                hout["dv"], hout["doff"], arena)
        torch.cuda.synchronize()
        assert torch.equal(hout["out"], out_d.cpu()) and torch.equal(hout["lse"], lse_d.cpu())
        assert torch.equal(hout["dq"], g_d[0].cpu()) and torch.equal(hout["doff"], g_d[3].cpu())
        for got, ref in ((hout["dk"], g_d[1]), (hout["dv"], g_d[2])):
            ref = ref.cpu().float()
            assert float((got.float() - ref).abs().max()) <= 2e-2 * float(ref.abs().max())
        for z in hout.values():
            z.fill_(float("nan"))


@pytest.mark.parametrize("dtype,shape", [(BF16, (19, 9, 10, 2, 128)), (F32, (6, 10, 12, 3, 64)), (BF16, (1, 7, 9, 2, 64))])
def test_pipelined_host_steps_match_the_device_entry_points(dtype, shape):
    """A sequence of dsa3d_step_host_pipelined calls on one arena - different inputs per step,
    each with its own host buffers - queued without waiting, then one flush: every step's results
    must equal dsa3d_forward + dsa3d_backward on its own inputs (the next call's uploads overlap
    this call's kernels, so a missing ordering between calls shows up as another step's data).
    Then a call with another shape on the same arena (which must wait for the whole previous
    call), and the plain entry point after pipelined ones."""
    window = (3, 3, 3)
    pin = lambda z: z.clone().pin_memory()

    def make(shape_, seed):
        q, k, v, off, dout = small_problem(*shape_, window, dtype, 1.3, seed)
        dims = tuple(q.shape)
        dev = [z.cuda() for z in (q, k, v, off, dout)]
        out_d, lse_d = pu.gpu_forward(*dev[:4], dims, window)
        g_d = pu.gpu_backward(*dev[:4], lse_d, dev[4], dims, window)
        hout = {n: torch.full_like(q, float("nan")).pin_memory() for n in ("out", "dq", "dk", "dv")}
        hout["lse"] = torch.full(dims[:4], float("nan")).pin_memory()
        hout["doff"] = torch.full_like(off, float("nan")).pin_memory()
        return dims, [pin(z) for z in (q, k, v, off, dout)], hout, (out_d.cpu(), lse_d.cpu(), [g.cpu() for g in g_d])

    def check(hout, ref):
        out_d, lse_d, g_d = ref
        assert torch.equal(hout["out"], out_d) and torch.equal(hout["lse"], lse_d)
        assert torch.equal(hout["dq"], g_d[0]) and torch.equal(hout["doff"], g_d[3])
        for got, r in ((hout["dk"], g_d[1]), (hout["dv"], g_d[2])):
            assert float((got.float() - r.float()).abs().max()) <= 2e-2 * float(r.float().abs().max())

    other = (shape[0] + 2, shape[1], shape[2] + 1, shape[3], shape[4])
    steps = [make(shape, 600 + i) for i in range(4)] + [make(other, 610)] + [make(shape, 611)]
    nbytes = max(binding.dsa3d_step_host_arena_bytes(*st[0], window, dtype) for st in steps)
    arena = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for dims, hin, hout, _ in steps:
        binding.dsa3d_step_host_pipelined(*hin, *dims, window, hout["out"], hout["lse"], hout["dq"], hout["dk"],
                                          hout["dv"], hout["doff"], arena)
    binding.dsa3d_step_host_flush()
    torch.cuda.synchronize()
    for _, _, hout, ref in steps:
        check(hout, ref)
    # the plain entry point right after pipelined calls, without a flush in between
    dims, hin, hout, ref = make(shape, 620)
    binding.dsa3d_step_host_pipelined(*steps[0][1], *steps[0][0], window, *(steps[0][2][n] for n in
                                      ("out", "lse", "dq", "dk", "dv", "doff")), arena)
    binding.dsa3d_step_host(*hin, *dims, window, hout["out"], hout["lse"], hout["dq"], hout["dk"], hout["dv"],
                            hout["doff"], arena)
    torch.cuda.synchronize()
    check(hout, ref)
    check(steps[0][2], steps[0][3])


def test_pipelined_host_steps_with_transfers_long_enough_to_overlap():
    """Three pipelined steps with different inputs at a size where each transfer and each kernel
    takes of the order of a millisecond (40 MB per tensor, 8 slabs), so that uploads of step i+1
    and downloads of step i really run beside kernels: per-query results must still be bitwise
    those of the device entry points."""
    shape, window = (16, 40, 60, 4, 128), (3, 3, 3)
    T, H, W, heads, d = shape
    n = T * H * W * heads
    steps = []
    for i in range(3):
        q, k, v, dout = (inputs.normal(shape, 630 + i, j, 1.0, BF16) for j in range(4))
        off = inputs.normal((T, H, W, heads, 27, 3), 630 + i, 4, 1.5, F32)
        dev = [z.cuda() for z in (q, k, v, off, dout)]
        out_d, lse_d = pu.gpu_forward(*dev[:4], shape, window)
        g_d = pu.gpu_backward(*dev[:4], lse_d, dev[4], shape, window)
        hout = {nm: torch.full(shape, float("nan"), dtype=BF16).pin_memory() for nm in ("out", "dq", "dk", "dv")}
        hout["lse"] = torch.full(shape[:4], float("nan")).pin_memory()
        hout["doff"] = torch.full(off.shape, float("nan")).pin_memory()
        steps.append(([z.pin_memory() for z in (q, k, v, off, dout)], hout,
                      (out_d.cpu(), lse_d.cpu(), [g.cpu() for g in g_d])))
        del dev, out_d, lse_d, g_d
    arena = torch.empty(binding.dsa3d_step_host_arena_bytes(*shape, window, BF16), dtype=torch.uint8, device="cuda")
    for rounds in range(2):                                   # the second round reuses events and both K/V buffers
        for hin, hout, _ in steps:
            binding.dsa3d_step_host_pipelined(*hin, *shape, window, hout["out"], hout["lse"], hout["dq"], hout["dk"],
                                              hout["dv"], hout["doff"], arena)
        binding.dsa3d_step_host_flush()
        torch.cuda.synchronize()
        for _, hout, (out_d, lse_d, g_d) in steps:
            assert torch.equal(hout["out"], out_d) and torch.equal(hout["lse"], lse_d)
            assert torch.equal(hout["dq"], g_d[0]) and torch.equal(hout["doff"], g_d[3])
            for got, r in ((hout["dk"], g_d[1]), (hout["dv"], g_d[2])):
                assert float((got.float() - r.float()).abs().max()) <= 2e-2 * float(r.float().abs().max())
            for z in hout.values():
                z.fill_(float("nan"))


@pytest.mark.parametrize("dtype,d", [(BF16, 128), (BF16, 64), (F32, 32)])
def test_integer_positions_mixed_with_real_ones(dtype, d):
    """The forward takes chunks of samples that all sit on grid positions through a batched
    one-row-per-sample path; the choice is per chunk and per warp, so mix the cases: integer
    offsets for the first 16 window cells only, and integer offsets for every other query."""
    q, k, v, off, dout = small_problem(4, 9, 11, 2, d, (3, 3, 3), dtype, 1.4, 70)
    ints = inputs.uniform_int(off.shape, 71, 3, -2, 2, torch.float32)
    a = off.clone()
    a[..., :16, :] = ints[..., :16, :]
    pu.full_parity(q, k, v, a, dout, (3, 3, 3))
    b = off.clone().view(-1, 2, 27, 3)
    b[0::2] = ints.view(-1, 2, 27, 3)[0::2]
    pu.full_parity(q, k, v, b.view_as(off), dout, (3, 3, 3))


# ------------------------------------------------------------------------ batched forms

def test_batched_entry_points_equal_one_call_per_video():
    """Two different videos stored back to back must come out exactly as from two single
    calls (per-query results bitwise; dk/dv up to the order of their atomic sums)."""
    vids = [small_problem(4, 8, 10, 2, 64, (3, 3, 3), BF16, 1.2, seed) for seed in (80, 81)]
    dims, win = (4, 8, 10, 2, 64), (3, 3, 3)
    cat = [torch.stack([vids[0][i], vids[1][i]]).cuda() for i in range(5)]       # q, k, v, off, dout
    out = torch.empty_like(cat[0])
    lse = torch.empty(2, *dims[:4], dtype=torch.float32, device="cuda")
    binding.dsa3d_forward_batch(*cat[:4], 2, *dims, win, out, lse)
    dq, dk, dv = (torch.full_like(cat[0], float("nan")) for _ in range(3))
    doff = torch.full_like(cat[3], float("nan"))
    ws = torch.empty(binding.dsa3d_backward_workspace_bytes(*dims, win, BF16), dtype=torch.uint8, device="cuda")
    binding.dsa3d_backward_batch(*cat[:4], lse, cat[4], 2, *dims, win, dq, dk, dv, doff, ws)
    torch.cuda.synchronize()
    for b in range(2):
        single = [z.cuda() for z in vids[b]]
        o1, l1 = pu.gpu_forward(*single[:4], dims, win)
        g1 = pu.gpu_backward(*single[:4], l1, single[4], dims, win)
        assert torch.equal(out[b], o1) and torch.equal(lse[b], l1)
        assert torch.equal(dq[b], g1[0]) and torch.equal(doff[b], g1[3])
        for got, ref in ((dk[b], g1[1]), (dv[b], g1[2])):
            assert float((got.float() - ref.float()).abs().max()) <= 2e-2 * float(ref.float().abs().max())
    # and the second video of the batch against the oracle directly
    import oracle
    qh, kh, vh, offh, douth = vids[1]
    o_ref, l_ref = oracle.forward(qh, kh, vh, offh, *dims, win)
    refs = oracle.backward(qh, kh, vh, offh, douth, *dims, win)
    pu.assert_close("batch out", out[1], o_ref, BF16)
    pu.assert_close("batch lse", lse[1], l_ref, BF16)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), (dq[1], dk[1], dv[1], doff[1]), refs):
        pu.assert_close("batch " + name, got, ref, BF16, backward=True)


# ----------------------------------------------------------------- stays inside its buffers

@pytest.mark.parametrize("dtype", [BF16, F32])
def test_nothing_is_written_outside_the_output_buffers(dtype):
    """Every output and the workspace are carved out of one arena with 4 KiB guard bands
    between them; after a forward and a backward on a ragged problem with many samples
    outside the grid the guard bands must still hold their pattern."""
    q, k, v, off, dout = small_problem(5, 7, 9, 3, 64, (3, 3, 3), dtype, 2.5, 90)
    dims, win = tuple(q.shape), (3, 3, 3)
    dev = [z.cuda() for z in (q, k, v, off, dout)]
    elt = q.element_size()
    n_rows, n_off, n_lse = q.numel() * elt, off.numel() * 4, q.numel() // dims[4] * 4
    ws_bytes = max(binding.dsa3d_backward_workspace_bytes(*dims, win, dtype), 16)
    sizes = {"out": n_rows, "lse": n_lse, "dq": n_rows, "dk": n_rows, "dv": n_rows, "doff": n_off, "ws": ws_bytes}
    guard, at, spans = 4096, 4096, {}
    for name, nbytes in sizes.items():
        spans[name] = (at, nbytes)
        at += (nbytes + 255) // 256 * 256 + guard
    arena = torch.full((at,), 0xA5, dtype=torch.uint8, device="cuda")

    def view(name, like_dtype, shape):
        start, nbytes = spans[name]
        return arena[start:start + nbytes].view(like_dtype).view(shape)

    out, lse = view("out", dtype, dims), view("lse", torch.float32, dims[:4])
    dq, dk, dv = (view(n, dtype, dims) for n in ("dq", "dk", "dv"))
    doff, ws = view("doff", torch.float32, off.shape), view("ws", torch.uint8, (ws_bytes,))
    binding.dsa3d_forward(*dev[:4], *dims, win, out, lse)
    binding.dsa3d_backward(*dev[:4], lse, dev[4], *dims, win, dq, dk, dv, doff, ws)
    torch.cuda.synchronize()
    inside = torch.zeros(at, dtype=torch.bool, device="cuda")
    for start, nbytes in spans.values():
        inside[start:start + nbytes] = True
    assert bool((arena[~inside] == 0xA5).all())
    o_ref, _ = oracle_forward(q, k, v, off, dims, win)
    pu.assert_close("out", out, o_ref, dtype)


def oracle_forward(q, k, v, off, dims, win):
    import oracle
    return oracle.forward(q, k, v, off, *dims, win)


# ------------------------------------------------------------- CUDA graph capture

@pytest.mark.parametrize("dtype", [BF16, F32])
def test_forward_and_backward_can_be_captured_in_a_cuda_graph(dtype):
    """Small problems are launch-bound, so a caller will want the step in a CUDA graph: the
    device entry points only enqueue work on the given stream (no allocation, no
    synchronisation), so forward + backward capture into one graph whose replays reproduce
    the eager results (dk/dv up to the order of their atomic sums)."""
    q, k, v, off, dout = small_problem(4, 9, 10, 2, 64, (3, 3, 3), dtype, 1.1, 95)
    dims = tuple(q.shape)
    T, H, W, heads, d = dims
    dev = [z.cuda() for z in (q, k, v, off, dout)]
    out_e, lse_e = pu.gpu_forward(*dev[:4], dims, (3, 3, 3))
    g_e = pu.gpu_backward(*dev[:4], lse_e, dev[4], dims, (3, 3, 3))
    out, lse = torch.empty_like(out_e), torch.empty_like(lse_e)
    dq, dk, dv, doff = (torch.empty_like(z) for z in g_e)
    ws = torch.empty(max(binding.dsa3d_backward_workspace_bytes(*dims, (3, 3, 3), dtype), 16), dtype=torch.uint8,
                     device="cuda")
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            binding.dsa3d_forward(*dev[:4], T, H, W, heads, d, (3, 3, 3), out, lse)
            binding.dsa3d_backward(*dev[:4], lse, dev[4], T, H, W, heads, d, (3, 3, 3), dq, dk, dv, doff, ws)
    for _ in range(2):
        for z in (out, lse, dq, dk, dv, doff):
            z.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, out_e) and torch.equal(lse, lse_e)
        assert torch.equal(dq, g_e[0]) and torch.equal(doff, g_e[3])
        for got, ref in ((dk, g_e[1]), (dv, g_e[2])):
            ref = ref.float()
            assert float((got.float() - ref).abs().max()) <= 2e-2 * float(ref.abs().max())


@pytest.mark.parametrize("dtype,shape", [(BF16, (19, 9, 10, 2, 128)), (F32, (11, 5, 6, 2, 32)), (BF16, (1, 7, 9, 2, 64))])
def test_forward_host_matches_the_device_forward(dtype, shape):
    """dsa3d_forward_host (host buffers in and out, slabs of frames pipelined over two side
    streams) returns exactly what dsa3d_forward returns on device buffers; twice in a row."""
    q, k, v, off, _ = small_problem(*shape, (3, 3, 3), dtype, 1.3, 61)
    dims = tuple(q.shape)
    out_d, lse_d = pu.gpu_forward(q.cuda(), k.cuda(), v.cuda(), off.cuda(), dims, (3, 3, 3))
    pin = lambda z: z.clone().pin_memory()
    hq, hk, hv, hoff = pin(q), pin(k), pin(v), pin(off)
    out_h = torch.full_like(q, float("nan")).pin_memory()
    lse_h = torch.full(dims[:4], float("nan")).pin_memory()
    arena = torch.empty(binding.dsa3d_forward_host_arena_bytes(*dims, (3, 3, 3), dtype), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        binding.dsa3d_forward_host(hq, hk, hv, hoff, *dims, (3, 3, 3), out_h, lse_h, arena)
        torch.cuda.synchronize()
        assert torch.equal(out_h, out_d.cpu()) and torch.equal(lse_h, lse_d.cpu())
        out_h.fill_(float("nan"))
        lse_h.fill_(float("nan"))
