"""The encode entry point that needs no scratch from the caller (``ciera_encode_noalloc``).

It exists for callers that own their parameter, cache and message buffers but cannot get one more
device allocation when they call (a memory pool that already holds the GPU, a hook that must not
stall the device, a plug-in without an allocator).  It must give exactly what ``ciera_encode``
gives -- messages, lengths, changed-block counts, sender cache, byte for byte -- also on a second
call, when its built-in scratch still holds the first call's contents.

Collected last (file name), so that a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.uint8).copy()).to(DEV)


@pytest.mark.parametrize("dtype,block", [("bf16", 512), ("fp32", 64)])
def test_noalloc_encode_equals_encode_on_two_calls_in_a_row(dtype, block):
    assert torch.cuda.is_available()
    from paper_2609_04609_b200 import ciera, runtime

    # multi-tile units (look-back across tiles uses the scratch), a ragged one and an empty one
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(1)] + [70001 * 16, 0, 33 * 16]
    ref = runtime.LayerCodec.from_tensors(sizes, 16, dtype, block, DEV)
    new = runtime.LayerCodec.from_tensors(sizes, 16, dtype, block, DEV)
    n = ref.weights_bytes // wl.VALUE_BYTES[dtype]
    traj = [_dev(wl.as_bits(w)) for w in wl.trajectory(n, dtype, 4711, 2, "clustered", f=0.3)]
    ref.init_caches(traj[0])
    new.init_caches(traj[0])
    for t in (1, 2):
        ciera.encode(ref.plan, traj[t], ref.sender_cache, ref.msg_send, ref.wire_bytes, ref.changed_blocks,
                     ref.workspace, ref.status)
        ciera.encode_noalloc(new.plan, traj[t], new.sender_cache, new.msg_send, new.wire_bytes, new.changed_blocks,
                             new.status)
        torch.cuda.synchronize()
        ref.check_status()
        new.check_status()
        assert torch.equal(ref.wire_bytes, new.wire_bytes), f"call {t}: lengths differ"
        assert torch.equal(ref.changed_blocks, new.changed_blocks), f"call {t}: changed-block counts differ"
        assert int(ref.changed_blocks.sum()) > 0
        assert torch.equal(ref.sender_cache, new.sender_cache), f"call {t}: sender caches differ"
        wire = ref.wire_bytes.cpu().numpy()
        a, b = ref.msg_send.cpu().numpy(), new.msg_send.cpu().numpy()
        for u, wb in zip(ref.units, wire):
            mo = int(u["msg_off"])
            assert np.array_equal(a[mo : mo + int(wb)], b[mo : mo + int(wb)]), f"call {t}: a message differs"
    # and the receiver reconstructs the weights from the no-scratch sender's messages
    new.transport()
    new.receiver_cache.copy_(ref.receiver_cache)
    ciera.cache_update(new.plan, new.receiver_cache, traj[1])
    new.decode()
    torch.cuda.synchronize()
    new.check_status()
    for u in new.units:
        lo, nb = int(u["weights_off"]), int(u["n_values"]) * wl.VALUE_BYTES[dtype]
        assert torch.equal(new.weights_out[lo : lo + nb], traj[2][lo : lo + nb])


def test_noalloc_encode_refuses_plans_beyond_its_scratch():
    from paper_2609_04609_b200 import ciera

    too_many = (ciera.NOALLOC_MAX_TILES + 1) * 8192
    units = np.array([(too_many, 0, 0, 0, ciera.message_capacity(too_many, ciera.BF16, 512))], dtype=wl.UNIT_DTYPE)
    plan = ciera.Plan(units, ciera.BF16, 512, DEV)
    assert plan.n_tiles == ciera.NOALLOC_MAX_TILES + 1
    dummy = torch.zeros(64, dtype=torch.uint8, device=DEV)
    wire = torch.zeros(1, dtype=torch.int64, device=DEV)
    chg = torch.zeros(1, dtype=torch.int32, device=DEV)
    with pytest.raises(ciera.CieraError) as e:
        ciera.encode_noalloc(plan, dummy, dummy, dummy, wire, chg)
    assert e.value.status == ciera.ERR_TOO_LARGE
    assert "built-in scratch" in str(e.value)
    torch.cuda.synchronize()
