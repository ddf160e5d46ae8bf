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

    # units of several tiles (runs of tiles hand their place in the payload on through the scratch), a ragged
    # one and an empty one; units of more than 32 tiles, whose tiles look back on each other, are in the test below
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


@pytest.mark.parametrize("dtype,block", [("bf16", 512), ("bf16", 4), ("fp16", 64), ("fp16", 2), ("fp32", 1)])
def test_noalloc_encode_with_long_units_equals_the_oracle(dtype, block):
    """Units of more than 32 tiles are spread over the thread blocks: their tiles find their place in the payload by
    a look-back over the status words in the built-in scratch, and the launch is a cooperative one.  The messages are
    compared with the CPU oracle's, byte for byte, on two calls; between them a call with a differently shaped plan
    leaves other contents in the scratch."""
    assert torch.cuda.is_available()
    from oracle import ciera_oracle as ora
    from paper_2609_04609_b200 import ciera, runtime

    code = ciera.DTYPE_CODES[dtype]
    vb = wl.VALUE_BYTES[dtype]
    wdt = np.uint32 if dtype == "fp32" else np.uint16
    sizes = [600_001, 8192 * 40, 131_072, 0, 33]
    new = runtime.LayerCodec.from_tensors(sizes, 1, dtype, block, DEV)
    assert max(int(u["n_values"]) for u in new.units) > 32 * 8192
    other = runtime.LayerCodec.from_tensors([r * c for r, c in wl.olmoe_layer_shapes(1)], 16, "bf16", 64, DEV)
    n = new.weights_bytes // vb
    traj = [wl.as_bits(w) for w in wl.trajectory(n, dtype, 815, 2, "clustered", f=0.3)]
    new.init_caches(_dev(traj[0]))
    caches = [ora.cache_init(traj[0][int(u["weights_off"]) // vb:][: int(u["n_values"])], int(u["n_values"]), code)
              for u in new.units]
    w_other = _dev(wl.as_bits(wl.init_weights(other.weights_bytes // 2, "bf16", wl.make_generator(3))))
    for t in (1, 2):
        ciera.encode_noalloc(new.plan, _dev(traj[t]), new.sender_cache, new.msg_send, new.wire_bytes, new.changed_blocks,
                             new.status)
        torch.cuda.synchronize()
        new.check_status()
        wire = new.wire_bytes.cpu().numpy()
        chg = new.changed_blocks.cpu().numpy()
        msgs = new.msg_send.cpu().numpy()
        cs = new.sender_cache.cpu().numpy()
        for i, u in enumerate(new.units):
            lo, nn, mo, co = int(u["weights_off"]) // vb, int(u["n_values"]), int(u["msg_off"]), int(u["cache_off"])
            m, wb, _, cb = ora.encode(traj[t][lo : lo + nn].astype(wdt), caches[i], code, block)
            assert int(wire[i]) == wb and int(chg[i]) == cb, f"call {t}, unit {i}: length / changed blocks"
            assert np.array_equal(msgs[mo : mo + wb], m), f"call {t}, unit {i}: message differs from the oracle's"
            assert np.array_equal(cs[co : co + nn], caches[i]), f"call {t}, unit {i}: sender cache differs"
        # another plan goes through the same built-in scratch in between
        ciera.encode_noalloc(other.plan, w_other, other.sender_cache, other.msg_send, other.wire_bytes,
                             other.changed_blocks, other.status)
        torch.cuda.synchronize()
        other.check_status()


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
