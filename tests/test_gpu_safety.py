"""Failure paths and memory discipline of the CUDA path, all provoked from the host.

* every device-side wait of the persistent kernels is bounded; the library's self-test runs both kinds
  of wait with a short limit on things that nobody completes and must come back with CIERA_ERR_TIMEOUT,
  a clean synchronise and a context in which the next ordinary step is still bit-exact;
* a reported message length that no sender step can produce (the stale word of a unit that an aborted
  encode never finished, a damaged word) must not make the transport or the entropy stage leave the
  unit's slot: CIERA_ERR_CORRUPT, neighbouring slots untouched;
* the guard bytes of tests/harness.py really notice a stray store.

Nothing here makes a kernel starve, trap or run at its production wait limits."""
import numpy as np
import pytest
import torch

from harness import Canaries, OracleTable, compare_caches, compare_recon, compare_step, guard, to_dev_bytes
from paper_2609_04609_b200 import workloads as wl

DEV = "cuda:0"


def test_uncovered_index_arithmetic():
    """(No GPU.)  The gap finder behind the guard bytes: units in any order, empty units, a tail."""
    off = np.array([64, 0, 32, 48], np.int64)
    length = np.array([10, 16, 0, 16], np.int64)
    got = Canaries._uncovered(off, length, 80)
    want = np.array(list(range(16, 48)) + list(range(74, 80)), np.int64)
    assert np.array_equal(got, want)
    assert Canaries._uncovered(np.zeros(0, np.int64), np.zeros(0, np.int64), 4).tolist() == [0, 1, 2, 3]
    with pytest.raises(AssertionError):
        Canaries._uncovered(np.array([0, 8], np.int64), np.array([16, 4], np.int64), 32)


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _clean_step_is_exact(rt, dtype=0, block=512):
    ciera, runtime = rt
    name = {0: "bf16", 1: "fp32", 2: "fp16"}[dtype]
    codec = guard(runtime.LayerCodec.from_tensors([3_000_000 + 5, 131_072, 70_001], 2, name, block, DEV, slack=256))
    table = OracleTable(codec.units, dtype, block, codec.cache_bytes, codec.msg_bytes)
    n = codec.weights_bytes // wl.VALUE_BYTES[name]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 99, 1, "clustered", f=0.3)]
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    table.init_caches(traj[0])
    codec.step(to_dev_bytes(traj[1], DEV))
    torch.cuda.synchronize()
    codec.check_status()
    exp = table.step(traj[1])
    compare_step(codec, exp, traj[1], "after the failure")
    compare_caches(codec, table, "after the failure")
    compare_recon(codec, exp, traj[1], dtype, "after the failure")


@pytest.mark.gpu
@pytest.mark.parametrize("max_polls", [8, 64])
def test_bounded_waits_run_out_and_the_context_stays_usable(rt, max_polls):
    ciera, _ = rt
    scratch = torch.full((2,), -1, dtype=torch.int64, device=DEV)  # the call clears the word it polls
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    report = torch.full((4,), -1, dtype=torch.int32, device=DEV)
    ciera.selftest_bounded_waits(max_polls, scratch, status, report)
    torch.cuda.synchronize()  # the kernel came back by itself
    assert int(status.item()) == ciera.ERR_TIMEOUT
    assert report.tolist() == [1, 1, 1, max_polls]
    assert int(scratch[1].item()) == -1  # only the polled word was touched
    # the status word is sticky: a second run does not overwrite an error that is already there
    status.fill_(ciera.ERR_CORRUPT)
    ciera.selftest_bounded_waits(max_polls, scratch, status, report)
    torch.cuda.synchronize()
    assert int(status.item()) == ciera.ERR_CORRUPT
    with pytest.raises(ciera.CieraError) as e:
        ciera.selftest_bounded_waits(0, scratch, status, report)
    assert e.value.status == ciera.ERR_INVALID_ARG
    with pytest.raises(ciera.CieraError):
        ciera.selftest_bounded_waits(1 << 20, scratch, status, report)  # not a way to stall the GPU
    _clean_step_is_exact(rt)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,block", [(0, 512), (1, 64), (0, 4), (2, 512), (2, 16)])
def test_transport_never_leaves_a_slot_on_an_impossible_length(rt, dtype, block):
    ciera, runtime = rt
    name = {0: "bf16", 1: "fp32", 2: "fp16"}[dtype]
    sizes = [70_001, 131_072, 40_000, 8192 * 3]
    codec = guard(runtime.LayerCodec.from_tensors(sizes, 1, name, block, DEV, slack=256))
    n = codec.weights_bytes // wl.VALUE_BYTES[name]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 7, 1, "adam")]
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    wd = to_dev_bytes(traj[1], DEV)
    codec.encode(wd)
    torch.cuda.synchronize()
    good = codec.wire_bytes.clone()
    # unit 1 (not the last one) claims more bytes than its slot holds; the other units are fine
    codec.wire_bytes[1] = int(codec.units[1]["msg_capacity"]) + 4096
    codec.msg_recv.fill_(0x3C)
    guard(codec)  # (the fill went over the guard bytes between the slots: arm them again)
    codec.transport()
    torch.cuda.synchronize()
    with pytest.raises(ciera.CieraError) as e:
        codec.check_status()
    assert e.value.status == ciera.ERR_CORRUPT
    codec.canaries.check("transport with an impossible length")
    recv, send = codec.msg_recv.cpu().numpy(), codec.msg_send.cpu().numpy()
    for i, u in enumerate(codec.units):
        mo, cap, used = int(u["msg_off"]), int(u["msg_capacity"]), int(good[i].item())
        if i == 1:
            assert np.all(recv[mo : mo + cap] == 0x3C), "the unit with the impossible length must move nothing"
        else:
            assert np.array_equal(recv[mo : mo + used], send[mo : mo + used]), f"unit {i} was not transported"
            assert np.all(recv[mo + used : mo + cap] == 0x3C), f"unit {i}: bytes past the reported length were written"
    # the entropy stage treats the same word as "nothing to code" and leaves the message alone
    before = codec.msg_send.clone()
    codec.status.zero_()
    codec.entropy_encode()
    torch.cuda.synchronize()
    mo, cap = int(codec.units[1]["msg_off"]), int(codec.units[1]["msg_capacity"])
    assert torch.equal(codec.msg_send[mo : mo + cap], before[mo : mo + cap])
    codec.canaries.check("entropy stage with an impossible length")
    _clean_step_is_exact(rt, dtype, block if block >= 16 else 512)


@pytest.mark.gpu
@pytest.mark.parametrize("block", [16, 512])
def test_entropy_stage_leaves_an_fp16_unit_alone_when_its_length_is_no_sum_of_block_sizes(rt, block):
    """fp16: the sender's entropy stage gets the number of five-bit symbols from the payload's length.  A length
    inside the slot that no set of changed blocks adds up to (here: one byte short) must make it leave the unit as
    it is; the other units are coded as usual."""
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors([70_001, 131_072, 40_000], 1, "fp16", block, DEV, slack=256))
    n = codec.weights_bytes // 2
    w = wl.as_bits(next(iter(wl.trajectory(n, "fp16", 12, 0, "adam"))))
    codec.init_caches(None)  # from empty caches: every block is sent
    codec.encode(to_dev_bytes(w, DEV))
    torch.cuda.synchronize()
    good = codec.wire_bytes.clone()
    codec.wire_bytes[1] = int(good[1].item()) - 1
    before = codec.msg_send.clone()
    codec.entropy_encode()
    torch.cuda.synchronize()
    codec.check_status()
    codec.canaries.check("entropy stage with a length that is no sum of block sizes")
    mo, cap = int(codec.units[1]["msg_off"]), int(codec.units[1]["msg_capacity"])
    assert torch.equal(codec.msg_send[mo : mo + cap], before[mo : mo + cap])
    assert int(codec.wire_bytes[1].item()) == int(good[1].item()) - 1
    for i in (0, 2):
        assert int(codec.wire_bytes[i].item()) < int(good[i].item())  # coded


@pytest.mark.gpu
def test_guard_bytes_notice_a_stray_store(rt):
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors([1000, 33, 70_001], 1, "bf16", 64, DEV, slack=256))
    assert codec.canaries.guarded_bytes() > 5 * 256
    codec.canaries.check("armed")
    end_of_first = int(codec.units[0]["cache_off"]) + 1000
    codec.allocations["receiver_cache"][end_of_first] = 0  # one byte past unit 0's cached exponents
    with pytest.raises(AssertionError, match="receiver_cache"):
        codec.canaries.check("planted")
    codec.allocations["receiver_cache"][end_of_first] = Canaries.PATTERN
    codec.allocations["wire_bytes"][len(codec.units)] = 0
    with pytest.raises(AssertionError, match="wire_bytes"):
        codec.canaries.check("planted")


@pytest.mark.gpu
def test_a_dirty_workspace_is_made_usable_again_by_workspace_init(rt):
    """The sender expects its scratch all zero.  What a kernel that gave up would leave behind is imitated from the
    host (the status words and counters overwritten with junk); `ciera_workspace_init` puts it right, and the next
    step is bit-exact and leaves the scratch all zero again -- also for a plan whose long unit makes the thread
    blocks look back on each other."""
    from harness import sender_scratch_is_clean

    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors([3_000_000 + 5, 131_072, 70_001], 2, "bf16", 512, DEV, slack=256))
    table = OracleTable(codec.units, 0, 512, codec.cache_bytes, codec.msg_bytes)
    n = codec.weights_bytes // 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 5150, 2, "clustered", f=0.3)]
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    table.init_caches(traj[0])
    for t in (1, 2):
        codec.workspace.fill_(0xEE)
        ciera.workspace_init(codec.plan, codec.workspace)
        assert sender_scratch_is_clean(codec)
        codec.step(to_dev_bytes(traj[t], DEV))
        torch.cuda.synchronize()
        codec.check_status()
        exp = table.step(traj[t])
        compare_step(codec, exp, traj[t], f"t={t}")
        compare_caches(codec, table, f"t={t}")  # (checks the scratch as well)
        compare_recon(codec, exp, traj[t], 0, f"t={t}")
