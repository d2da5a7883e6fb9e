"""dK/dV by key blocks on the tensor cores (DSA3D_KEY_BLOCKS=1): the coefficient matrices of a block of
256 keys against chunks of 32 queries, multiplied by tcgen05 in tf32, instead of the tile kernel's
binning.  Every gradient is compared with the CPU oracle element by element at the bf16 tolerance
(the coefficients lose the bits below 2^-10 relative on this path, q and dO none); per-query results
must not depend on the path at all."""
import pytest
import torch

import oracle
import parity_util as pu
from paper_2607_22696_b200 import binding, inputs
from test_gpu_parity import small_problem

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


@pytest.fixture(autouse=True)
def key_blocks(monkeypatch):
    monkeypatch.setenv("DSA3D_KEY_BLOCKS", "1")
    yield
    assert binding.dsa3d_device_timeout_flag() == 0


@pytest.mark.parametrize("shape,window,sigma", [
    ((5, 7, 9, 3, 64), (3, 3, 3), 1.0),          # one block per head, ragged everywhere
    ((9, 17, 19, 2, 128), (3, 3, 3), 2.0),       # several blocks per axis, offsets that reach the region's edge
    ((13, 9, 26, 1, 128), (3, 3, 3), 4.0),       # many corners beyond the region: the gather kernel's own scatter
    ((4, 8, 8, 2, 64), (2, 2, 2), 0.7),          # exactly one block, even window
    ((6, 10, 12, 2, 128), (1, 1, 1), 1.5),
    ((1, 1, 1, 1, 128), (3, 3, 3), 0.5),
    ((1, 9, 40, 2, 64), (3, 3, 3), 1.0),
    ((12, 1, 11, 2, 128), (3, 3, 3), 1.0),
])
def test_key_block_kernel_matches_the_oracle(shape, window, sigma):
    pu.full_parity(*small_problem(*shape, window, BF16, sigma, 900 + shape[0] + shape[2]), window)


@pytest.mark.parametrize("window", [(3, 5, 5), (3, 7, 7), (4, 8, 8)])
def test_windows_of_more_than_32_samples_take_several_passes(window):
    pu.full_parity(*small_problem(6, 11, 13, 2, 128, window, BF16, 1.5, 910), window)
    pu.full_parity(*small_problem(5, 9, 10, 2, 64, window, BF16, 0.3, 911), window)


def test_zero_integer_and_dead_offsets():
    """Zero offsets fill the central chunks' lists completely (every sample of a block's own queries
    touches the block); integer offsets leave corner weights of exactly 0 and 1; NaN, infinite and
    huge offsets give dead samples, which must reach neither kernel's scatter."""
    q, k, v, off, dout = small_problem(8, 12, 17, 2, 128, (3, 3, 3), BF16, 1.0, 920)
    pu.full_parity(q, k, v, torch.zeros_like(off), dout, (3, 3, 3))
    ioff = inputs.uniform_int(off.shape, 921, 3, -3, 3, F32)
    pu.full_parity(q, k, v, ioff, dout, (3, 3, 3))
    bad = off.clone()
    flat = bad.view(-1)
    flat[5::97] = float("nan")
    flat[11::89] = float("inf")
    flat[17::83] = -3.0e38
    pu.full_parity(q, k, v, bad, dout, (3, 3, 3))


def test_per_query_results_do_not_depend_on_the_path_and_dk_dv_agree(monkeypatch):
    q, k, v, off, dout = small_problem(10, 14, 18, 3, 128, (3, 3, 3), BF16, 2.0, 930)
    dims = tuple(q.shape)
    dev = [z.cuda() for z in (q, k, v, off, dout)]
    out, lse = pu.gpu_forward(*dev[:4], dims, (3, 3, 3))
    blocks = pu.gpu_backward(*dev[:4], lse, dev[4], dims, (3, 3, 3))
    monkeypatch.setenv("DSA3D_KEY_BLOCKS", "0")
    tiles = pu.gpu_backward(*dev[:4], lse, dev[4], dims, (3, 3, 3))
    assert torch.equal(blocks[0], tiles[0]) and torch.equal(blocks[3], tiles[3])      # dq, doffsets
    for a, b in ((blocks[1], tiles[1]), (blocks[2], tiles[2])):
        a, b = a.float(), b.float()
        step = (b.abs() * 2.0 ** -7).clamp_min(float(b.pow(2).mean().sqrt()) * 2.0 ** -7)    # one bf16 step
        assert bool(((a - b).abs() <= step).all())


@pytest.mark.parametrize("shape", [(19, 9, 10, 2, 128), (6, 10, 12, 3, 64)])
def test_host_step_in_slabs_of_frames(shape):
    """dsa3d_step_host walks the video in slabs of frames: each slab's key-block launch adds the
    contributions of that slab's queries only, to every block its frames can reach."""
    window = (3, 3, 3)
    q, k, v, off, dout = small_problem(*shape, window, BF16, 1.3, 940)
    dims = tuple(q.shape)
    pin = lambda z: z.clone().pin_memory()
    hin = [pin(z) for z in (q, k, v, off, dout)]
    hout = {n: torch.full_like(q, float("nan")).pin_memory() for n in ("out", "dq", "dk", "dv")}
    hout["lse"] = torch.full(dims[:4], float("nan")).pin_memory()
    hout["doff"] = torch.full_like(off, float("nan")).pin_memory()
    arena = torch.empty(binding.dsa3d_step_host_arena_bytes(*dims, window, BF16), dtype=torch.uint8, device="cuda")
    binding.dsa3d_step_host(*hin, *dims, window, hout["out"], hout["lse"], hout["dq"], hout["dk"], hout["dv"],
                            hout["doff"], arena)
    torch.cuda.synchronize()
    T, H, W, heads, d = dims
    refs = oracle.backward(q, k, v, off, dout, T, H, W, heads, d, window)
    for name, got, ref in zip(("dq", "dk", "dv", "doffsets"), (hout["dq"], hout["dk"], hout["dv"], hout["doff"]), refs):
        pu.assert_close(name, got, ref, BF16, backward=True)
