"""Head sharding on one GPU: a problem is cut along the head axis with the helpers of
`sharding`, every shard runs dsa3d_forward + dsa3d_backward as a call of its own (one after
the other on the same device, the way the ranks of a multi-GPU job would each run theirs),
the pieces are put back together, and the result is compared with the unsharded call and
with the CPU oracle.  Heads never exchange anything inside the operator (the Formulation
gives every head its own offsets and its own q/k/v channels), so the per-query tensors must
agree bit for bit; dk/dv are sums of atomics whose order differs between the two runs."""
import pytest
import torch

import oracle
import parity_util as pu
from paper_2607_22696_b200 import inputs, sharding

pytestmark = pytest.mark.gpu


def _run(t, dims, window):
    out, lse = pu.gpu_forward(t["q"], t["k"], t["v"], t["offsets"], dims, window)
    dq, dk, dv, doff = pu.gpu_backward(t["q"], t["k"], t["v"], t["offsets"], lse, t["dout"], dims, window)
    return {"out": out, "lse": lse, "dq": dq, "dk": dk, "dv": dv, "doffsets": doff}


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 128), (torch.float32, 32)])
def test_head_shards_reassemble_to_the_unsharded_result_and_the_oracle(world, dtype, d):
    T, H, W, heads, window = 5, 9, 12, 5, (3, 3, 3)           # 5 heads over 2 or 3 shards: uneven split
    wl = inputs.Workload("shard", T, H, W, heads, d, window, dtype, 1.3, 310 + world)
    host = inputs.make_inputs(wl, "cpu", with_dout=True)
    full = {n: z.cuda() for n, z in host.items()}
    whole = _run(full, (T, H, W, heads, d), window)

    parts = []
    for rank in range(world):
        lo, hi = sharding.head_range(heads, world, rank)
        mine = {n: sharding.shard_heads(z, world, rank) for n, z in full.items()}
        assert mine["q"].shape[3] == hi - lo and mine["offsets"].shape[3] == hi - lo
        parts.append(_run(mine, (T, H, W, hi - lo, d), window))
    joined = {n: sharding.unshard_heads([p[n] for p in parts]) for n in whole}

    for n in ("out", "lse", "dq", "doffsets"):                # per-query tensors: deterministic
        assert torch.equal(joined[n], whole[n]), n
    for n in ("dk", "dv"):
        a, b = joined[n].float(), whole[n].float()
        assert float((a - b).abs().max()) <= 1e-2 * float(b.abs().max()), n

    o_ref, l_ref = oracle.forward(host["q"], host["k"], host["v"], host["offsets"], T, H, W, heads, d, window)
    refs = oracle.backward(host["q"], host["k"], host["v"], host["offsets"], host["dout"], T, H, W, heads, d, window)
    pu.assert_close("out", joined["out"], o_ref, dtype)
    pu.assert_close("lse", joined["lse"], l_ref, dtype)
    for n, ref in zip(("dq", "dk", "dv", "doffsets"), refs):
        pu.assert_close(n, joined[n], ref, dtype, backward=True)
