"""Parity of the CUDA path (through the C ABI) with the CPU oracle: tolerance 0.

Messages (bitmap, pads, sign-plus-mantissa, payload), per-unit byte counts and changed-block
counts, both caches and the reconstructed weights are compared byte for byte on the same
seeded inputs, over several tiles, ragged tails and every supported block size."""
import numpy as np
import pytest
import torch

from harness import OracleTable, compare_caches, compare_recon, compare_step, guard, to_dev_bytes
from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
WDT = {0: np.uint16, 1: np.uint32}
NAME = {0: "bf16", 1: "fp32"}


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _make(rt, sizes, n_shards, dtype, block):
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors(sizes, n_shards, NAME[dtype], block, DEV, slack=256))
    table = OracleTable(codec.units, dtype, block, codec.cache_bytes, codec.msg_bytes)
    n_flat = codec.weights_bytes // (2 if dtype == 0 else 4)
    return codec, table, n_flat


def _run_trajectory(rt, codec, table, traj, dtype, zero_cache=False, label=""):
    w0 = traj[0]
    if zero_cache:
        codec.init_caches(None)
        table.init_caches(None)
    else:
        codec.init_caches(to_dev_bytes(w0, DEV))
        table.init_caches(w0)
    compare_caches(codec, table, label + " init")
    stats = []
    for t, w in enumerate(traj[1:], 1):
        wd = to_dev_bytes(w, DEV)
        codec.step(wd)
        torch.cuda.synchronize()
        codec.check_status()
        exp = table.step(w)
        wire, chg = compare_step(codec, exp, w, f"{label} t={t}")
        compare_caches(codec, table, f"{label} t={t}")
        compare_recon(codec, exp, w, dtype, f"{label} t={t}")
        stats.append((int(chg.sum()), codec.n_blocks()))
    return stats


def test_config1_tiny_trajectory(rt):
    """1024x512 bf16, 4 row-block shards, 3 Gaussian steps, B = 512."""
    codec, table, n = _make(rt, [1024 * 512], 4, 0, 512)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 1235, 3, "gaussian")]
    stats = _run_trajectory(rt, codec, table, traj, 0, label="config1")
    assert all(c > 0 for c, _ in stats)
    # the paper's byte count from the device-reported lengths equals the oracle's
    assert codec.paper_bytes() > 0


@pytest.mark.parametrize("dtype,model,kw", [(0, "adam", {}), (0, "clustered", {"f": 0.22}), (1, "adam", {}),
                                            (1, "clustered", {"f": 0.22})])
def test_reduced_moe_layer(rt, dtype, model, kw):
    """4 experts x (2048x1024, 2048x1024, 1024x2048), 16 shards: the unit shape of the OLMoE
    configs (131 072 values = 16 tiles = 256 blocks per unit)."""
    shapes = wl.olmoe_layer_shapes(4)
    codec, table, n = _make(rt, [r * c for r, c in shapes], 16, dtype, 512)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 1236 + dtype, 2, model, **kw)]
    stats = _run_trajectory(rt, codec, table, traj, dtype, label=f"moe-{NAME[dtype]}-{model}")
    if model == "clustered":
        q = stats[-1][0] / stats[-1][1]
        assert 0.15 < q < 0.30


RAGGED = [0, 1, 15, 16, 17, 31, 33, 511, 512, 513, 1000, 4095, 4097, 8191, 8192, 8193, 8208, 16383, 16385, 20000,
          0, 70001, 131072 + 7]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block", [1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096])
def test_ragged_units_every_block_size(rt, dtype, block):
    """Units shorter than a block, not multiples of 16 / of the block / of the tile, empty units;
    random bit patterns (NaN, Inf, subnormals, both zeros included)."""
    codec, table, n = _make(rt, RAGGED, 1, dtype, block)
    rng = np.random.default_rng(100 * dtype + block)
    hi = 1 << (16 if dtype == 0 else 32)
    w0 = rng.integers(0, hi, n, dtype=np.uint64).astype(WDT[dtype])
    w1 = w0.copy()
    flip = rng.random(n) < 0.01
    w1[flip] = rng.integers(0, hi, int(flip.sum()), dtype=np.uint64).astype(WDT[dtype])
    w2 = w1.copy()  # nothing changes
    w3 = rng.integers(0, hi, n, dtype=np.uint64).astype(WDT[dtype])  # nearly everything changes
    _run_trajectory(rt, codec, table, [w0, w1, w2, w3], dtype, label=f"ragged-{NAME[dtype]}-B{block}")


@pytest.mark.parametrize("dtype", [0, 1])
def test_zero_initialised_caches(rt, dtype):
    codec, table, n = _make(rt, [5000, 8192 * 3 + 5], 2, dtype, 64)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 77, 2, "adam")]
    _run_trajectory(rt, codec, table, traj, dtype, zero_cache=True, label="zero-cache")


@pytest.mark.parametrize("block,c,seg", [(512, 0.001, 0), (64, 0.01, 0), (4096, 0.3, 4096), (2048, 0.0005, 0),
                                         (1024, 0.5, 0), (16, 0.05, 0), (1, 0.03, 0), (2, 0.0005, 0), (4, 0.4, 0),
                                         (8, 0.01, 0), (1, 0.6, 0)])
def test_long_units_look_back_over_many_tiles(rt, block, c, seg):
    """One unit of ~3 M values = 367 tiles (more than ten look-back windows) and a second,
    shorter one; exponent changes injected at an exact rate."""
    codec, table, n = _make(rt, [3_000_000 + 123, 600_000], 1, 0, block)
    gen = wl.make_generator(4242 + block)
    w0 = wl.init_weights(n, "bf16", gen)
    w1 = wl.inject_exponent_changes(w0, gen, c, seg)
    w2 = wl.inject_exponent_changes(w1, gen, c, seg)
    _run_trajectory(rt, codec, table, [wl.as_bits(w) for w in (w0, w1, w2)], 0, label=f"long-B{block}")


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block", [1, 2, 4, 8])
def test_small_blocks_on_a_reduced_moe_layer(rt, dtype, block):
    """Blocks of 1 to 8 values (B = 1: one bitmap bit per value, the payload holds exactly the
    exponents that changed) on 2 experts x 3 matrices x 4 shards plus ragged dense tensors, under the
    Adam-like update (a few per cent of the exponents change) and from zero caches."""
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(2)] + [70_001, 8192, 8191, 17, 0, 40_000]
    codec, table, n = _make(rt, sizes, 4, dtype, block)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 500 + block, 3, "adam")]
    stats = _run_trajectory(rt, codec, table, traj, dtype, label=f"small-{NAME[dtype]}-B{block}")
    assert 0 < stats[-1][0] < stats[-1][1]
    _run_trajectory(rt, codec, table, traj[:2], dtype, zero_cache=True, label=f"small-zero-{NAME[dtype]}-B{block}")


def test_change_rate_sweep_mixed_shapes(rt):
    """Fine-grained experts (2048x512) and small dense tensors, 8 / 64 shards, exponent change
    rates 0.1 %, 1 %, 10 %, 50 %."""
    shapes = [r * c for r, c in wl.fine_grained_layer_shapes(2)] + wl.dense_tensor_sizes()[:5]
    for n_shards, c in [(8, 0.001), (64, 0.01), (32, 0.1), (16, 0.5)]:
        codec, table, n = _make(rt, shapes, n_shards, 0, 512)
        gen = wl.make_generator(9000 + n_shards)
        w0 = wl.init_weights(n, "bf16", gen)
        w1 = wl.inject_exponent_changes(w0, gen, c)
        stats = _run_trajectory(rt, codec, table, [wl.as_bits(w0), wl.as_bits(w1)], 0, label=f"sweep-{n_shards}-{c}")
        assert stats[0][0] > 0


@pytest.mark.parametrize("dtype,block", [(0, 64), (0, 512), (0, 1), (0, 4096), (1, 8), (1, 256)])
def test_repeated_runs_are_identical(rt, dtype, block):
    """Same input three times from the same start state: every output byte equal (no order dependence in the
    look-back between thread blocks, in the hand-off between runs of tiles or in the dynamic hand-out of work).
    The table has a unit whose tiles are spread over the thread blocks, units worked through in runs, short ones."""
    ciera, runtime = rt
    outs = []
    for _ in range(3):
        codec, table, n = _make(rt, [2_000_000, 300_000, 131072, 8192 * 13 - 3, 70_001], 2, dtype, block)
        gen = wl.make_generator(31337)
        w0 = wl.init_weights(n, NAME[dtype], gen)
        w1 = wl.step_adam_like(w0, gen) if block < 256 else wl.step_clustered(w0, gen, f=0.4)
        codec.init_caches(to_dev_bytes(wl.as_bits(w0), DEV))
        codec.msg_send.zero_()
        codec.msg_recv.zero_()
        codec.step(to_dev_bytes(wl.as_bits(w1), DEV))
        torch.cuda.synchronize()
        codec.check_status()
        wire = codec.wire_bytes.cpu().numpy()
        ms = codec.msg_send.cpu().numpy()
        used = np.concatenate([ms[int(u["msg_off"]) : int(u["msg_off"]) + int(wb)] for u, wb in zip(codec.units, wire)])
        outs.append((wire.copy(), used, codec.changed_blocks.cpu().numpy().copy(), codec.sender_cache.cpu().numpy().copy(),
                     codec.receiver_cache.cpu().numpy().copy(), codec.weights_out.cpu().numpy().copy()))
    for other in outs[1:]:
        for a, b in zip(outs[0], other):
            assert np.array_equal(a, b)


def test_length_check_flags_a_corrupted_message(rt):
    """A failure made on the host: the reported length is altered after the encode, the receiver's
    check raises CIERA_ERR_CORRUPT in the status word and the context stays usable."""
    ciera, runtime = rt
    codec, table, n = _make(rt, [50000], 1, 0, 512)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 5, 1, "adam")]
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    wd = to_dev_bytes(traj[1], DEV)
    codec.encode(wd)
    codec.transport()
    codec.wire_bytes += 512
    codec.decode()
    torch.cuda.synchronize()
    with pytest.raises(ciera.CieraError) as e:
        codec.check_status()
    assert e.value.status == ciera.ERR_CORRUPT
    # the device is still fine: a clean step afterwards succeeds
    codec.status.zero_()
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    codec.step(wd)
    torch.cuda.synchronize()
    codec.check_status()
    out = codec.weights_out.cpu().numpy().view(np.uint16)[:50000]
    assert np.array_equal(out, traj[1][:50000])


def test_cache_update_and_bad_arguments(rt):
    ciera, runtime = rt
    codec, table, n = _make(rt, [10000, 33], 1, 1, 128)
    w = wl.as_bits(wl.init_weights(n, "fp32", wl.make_generator(1)))
    wd = to_dev_bytes(w, DEV)
    ciera.cache_update(codec.plan, codec.sender_cache, wd)
    ciera.cache_update(codec.plan, codec.receiver_cache, wd)
    table.init_caches(w)
    torch.cuda.synchronize()
    compare_caches(codec, table, "cache_update")
    with pytest.raises(ciera.CieraError) as e:
        ciera.cache_update(codec.plan, codec.sender_cache, None)
    assert e.value.status == ciera.ERR_INVALID_ARG
    with pytest.raises(ciera.CieraError) as e:
        ciera.encode(codec.plan, wd[1:], codec.sender_cache, codec.msg_send, codec.wire_bytes, codec.changed_blocks,
                     codec.workspace, codec.status)
    assert e.value.status == ciera.ERR_MISALIGNED
    with pytest.raises(ciera.CieraError) as e:
        ciera.decode(codec.plan, None, codec.receiver_cache, codec.weights_out)
    assert e.value.status == ciera.ERR_INVALID_ARG


def test_pipelined_stack_equals_serial(rt):
    """Two-stream layer pipeline (encode/transport of layer l+1 beside decode of layer l) gives
    byte-identical results to running the layers one after the other."""
    ciera, runtime = rt
    n_layers = 4
    shapes = [r * c for r, c in wl.olmoe_layer_shapes(2)]
    results = []
    for mode in ("serial", "pipelined"):
        layers, ws0, ws1 = [], [], []
        for l in range(n_layers):
            codec = runtime.LayerCodec.from_tensors(shapes, 16, "bf16", 512, DEV)
            n = codec.weights_bytes // 2
            gen = wl.make_generator(500 + l)
            w0 = wl.init_weights(n, "bf16", gen)
            w1 = wl.step_clustered(w0, gen, f=0.3)
            layers.append(codec)
            ws0.append(to_dev_bytes(wl.as_bits(w0), DEV))
            ws1.append(to_dev_bytes(wl.as_bits(w1), DEV))
            codec.init_caches(ws0[-1])
        torch.cuda.synchronize()
        if mode == "serial":
            for l in range(n_layers):
                layers[l].step(ws1[l])
        else:
            s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
            runtime.pipelined_step(layers, ws1, [None] * n_layers, s1, s2)
        torch.cuda.synchronize()
        for l in range(n_layers):
            layers[l].check_status()
            assert torch.equal(layers[l].weights_out[: ws1[l].numel()], ws1[l])
        results.append([(c.wire_bytes.cpu(), c.sender_cache.cpu(), c.receiver_cache.cpu(), c.weights_out.cpu())
                        for c in layers])
    for a, b in zip(*results):
        for x, y in zip(a, b):
            assert torch.equal(x, y)


@pytest.mark.parametrize("sizes,dtype,block", [([3_000_005, 131_072, 70_001], 0, 512), ([200_000, 5, 8192 * 3], 0, 4),
                                               ([131_072, 70_001], 1, 64), ([131_072, 70_001], 2, 512)])
def test_steps_replayed_from_a_cuda_graph(rt, sizes, dtype, block):
    """A whole step (sender, transport, receiver) is a handful of kernel launches that read their sizes on the
    device and leave the scratch as they found it, so it can be captured once in a CUDA graph and replayed on new
    weights in the same buffer.  Every replay must equal the oracle's step bit for bit, with a long unit
    (cooperative launch, prefix kernel) in the table as well."""
    ciera, runtime = rt
    name = {0: "bf16", 1: "fp32", 2: "fp16"}[dtype]
    codec = guard(runtime.LayerCodec.from_tensors(sizes, 2, name, block, DEV, slack=256))
    table = OracleTable(codec.units, dtype, block, codec.cache_bytes, codec.msg_bytes)
    n = codec.weights_bytes // wl.VALUE_BYTES[name]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 321 + block, 4, "clustered", f=0.3)]
    codec.init_caches(to_dev_bytes(traj[0], DEV))
    table.init_caches(traj[0])
    w_in = to_dev_bytes(traj[1], DEV).clone()
    codec.step(w_in)  # outside the capture first: the first calls query occupancy and set kernel attributes
    torch.cuda.synchronize()
    codec.check_status()
    compare_step(codec, table.step(traj[1]), traj[1], "eager")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=torch.cuda.Stream()):
        codec.step(w_in)
    for t in (2, 3, 4):
        w_in.copy_(to_dev_bytes(traj[t], DEV))
        graph.replay()
        torch.cuda.synchronize()
        codec.check_status()
        exp = table.step(traj[t])
        compare_step(codec, exp, traj[t], f"replay t={t}")
        compare_caches(codec, table, f"replay t={t}")
        compare_recon(codec, exp, traj[t], dtype, f"replay t={t}")


@pytest.mark.parametrize("dtype,block", [(0, 1), (0, 8), (0, 512), (2, 1), (2, 4), (2, 64), (1, 2), (1, 512)])
def test_every_pattern_against_every_cached_exponent(rt, dtype, block):
    """The complete per-value map on the GPU: every 16-bit pattern of bf16 and fp16 (zeros, subnormals, infinities,
    NaNs with every payload) against every value the cached exponent can have (256 / 32) -- 16.7 M / 2.1 M values in
    one unit, cache rows shuffled so that changed and unchanged blocks mix; for fp32 every exponent field x both
    signs x 4096 mantissas (the extreme ones among them) against eight cached exponents.  Message, length, count,
    caches and output against the oracle."""
    ciera, runtime = rt
    from oracle import ciera_oracle as ora

    rng = np.random.default_rng(1000 + 16 * dtype + block)
    if dtype == 1:
        mant = np.unique(np.concatenate([[0, 1, 2, (1 << 23) - 1, 1 << 22], rng.integers(0, 1 << 23, 4091)])).astype(np.uint32)
        pat = (np.arange(512, dtype=np.uint32)[:, None] << 23 | mant[None, :]).reshape(-1)  # sign and exponent x mantissas
        cached = np.array([0, 1, 126, 127, 128, 254, 255, 77], np.uint8)
        name, wdt = "fp32", np.uint32
        own = ((pat >> 23) & 0xFF).astype(np.uint8)
    else:
        pat = np.arange(1 << 16, dtype=np.uint16)
        cached = np.arange(256 if dtype == 0 else 32, dtype=np.uint8)
        name, wdt = ("bf16", np.uint16) if dtype == 0 else ("fp16", np.uint16)
        own = ((pat >> 7) & 0xFF).astype(np.uint8) if dtype == 0 else ((pat >> 10) & 0x1F).astype(np.uint8)
    w = np.tile(pat, cached.size).astype(wdt)
    cache0 = np.repeat(cached, pat.size)
    # in half of the rows the cache already holds the value's own exponent for most values: unchanged blocks too
    keep = np.repeat(rng.random(cached.size) < 0.5, pat.size) & (rng.random(w.size) < 0.97)
    cache0 = np.where(keep, np.tile(own, cached.size), cache0).astype(np.uint8)
    n = w.size
    codec = guard(runtime.LayerCodec.from_tensors([n], 1, name, block, DEV, slack=256))
    assert len(codec.units) == 1
    u = codec.units[0]
    lo, mo, co = int(u["weights_off"]), int(u["msg_off"]), int(u["cache_off"])
    w_dev = torch.zeros(codec.weights_bytes, dtype=torch.uint8, device=DEV)
    w_dev[lo : lo + w.nbytes] = torch.from_numpy(w.view(np.uint8)).to(DEV)
    for cache in (codec.sender_cache, codec.receiver_cache):
        cache[co : co + n] = torch.from_numpy(cache0).to(DEV)
    codec.step(w_dev)
    torch.cuda.synchronize()
    codec.check_status()
    codec.canaries.check("every pattern")
    cache_s = cache0.copy()
    msg, wire, pay, chg = ora.encode(w, cache_s, dtype, block)
    assert int(codec.wire_bytes[0].item()) == wire and int(codec.changed_blocks[0].item()) == chg
    assert 0 < chg < -(-n // block) or block >= 64
    assert np.array_equal(codec.msg_send[mo : mo + wire].cpu().numpy(), msg)
    assert np.array_equal(codec.msg_recv[mo : mo + wire].cpu().numpy(), msg)
    cache_r = cache0.copy()
    out = ora.decode(msg, cache_r, dtype, block)
    assert np.array_equal(out, w)
    assert np.array_equal(codec.sender_cache[co : co + n].cpu().numpy(), cache_s)
    assert np.array_equal(codec.receiver_cache[co : co + n].cpu().numpy(), cache_r)
    assert np.array_equal(codec.weights_out[lo : lo + w.nbytes].cpu().numpy().view(wdt), w)


@pytest.mark.parametrize("dtype,block", [(0, 512), (1, 4), (2, 64)])
def test_resume_from_saved_caches_or_from_the_weights(rt, dtype, block):
    """The codec's only persistent state are the two exponent caches (and the sender's HashCache), plain buffers of
    the caller.  A run is resumed either by putting saved copies of them back into fresh buffers, or -- since
    after every step both caches hold exactly the exponents of the weights just sent -- by rebuilding them from
    those weights.  Both ways the next step is the one the uninterrupted run makes, bit for bit."""
    ciera, runtime = rt
    name = {0: "bf16", 1: "fp32", 2: "fp16"}[dtype]
    sizes = [300_001, 131_072, 70_001]

    def fresh():
        return guard(runtime.LayerCodec.from_tensors(sizes, 2, name, block, DEV, slack=256))

    first = fresh()
    table = OracleTable(first.units, dtype, block, first.cache_bytes, first.msg_bytes)
    n = first.weights_bytes // wl.VALUE_BYTES[name]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 77 + block, 3, "clustered", f=0.3)]
    first.init_caches(to_dev_bytes(traj[0], DEV))
    table.init_caches(traj[0])
    for t in (1, 2):
        first.step(to_dev_bytes(traj[t], DEV))
        torch.cuda.synchronize()
        first.check_status()
        compare_step(first, table.step(traj[t]), traj[t], f"t={t}")
    saved_s, saved_r = first.sender_cache.cpu(), first.receiver_cache.cpu()  # the checkpoint
    want = table.step(traj[3])  # what the uninterrupted run does next

    restored = fresh()
    restored.sender_cache.copy_(saved_s)
    restored.receiver_cache.copy_(saved_r)
    guard(restored)  # (the copies went over the guard bytes: arm them again)
    rebuilt = fresh()
    rebuilt.init_caches(to_dev_bytes(traj[2], DEV))
    for label, codec in (("saved caches", restored), ("caches rebuilt from the weights", rebuilt)):
        codec.step(to_dev_bytes(traj[3], DEV))
        torch.cuda.synchronize()
        codec.check_status()
        compare_step(codec, want, traj[3], label)
        compare_caches(codec, table, label)
        compare_recon(codec, want, traj[3], dtype, label)
    if block >= 16:  # the hashed sender resumes from a HashCache rebuilt from the weights of the last step sent
        hashed = fresh()
        hashed.init_hash_cache(to_dev_bytes(traj[2], DEV))
        hashed.encode_hashed(to_dev_bytes(traj[3], DEV))
        hashed.transport()
        torch.cuda.synchronize()
        hashed.check_status()
        compare_step(hashed, want, traj[3], "HashCache rebuilt from the weights")


@pytest.mark.parametrize("n_layers", [1, 3])
def test_pipeline_of_many_iterations_reuses_layer_buffers_safely(rt, n_layers):
    """Many iterations back to back on two streams, alternating between two iterates: with a single
    layer the next iteration's sender side would overwrite the message that is still being decoded
    unless it waits for that decode.  Every iteration must come out exact and with a clean status."""
    ciera, runtime = rt
    shapes = [r * c for r, c in wl.olmoe_layer_shapes(8)]
    layers, wa, wb = [], [], []
    for l in range(n_layers):
        codec = runtime.LayerCodec.from_tensors(shapes, 16, "bf16", 512, DEV)
        n = codec.weights_bytes // 2
        gen = wl.make_generator(700 + l)
        w0 = wl.init_weights(n, "bf16", gen)
        w1 = wl.step_clustered(w0, gen, f=0.3)
        layers.append(codec)
        wa.append(to_dev_bytes(wl.as_bits(w0), DEV))
        wb.append(to_dev_bytes(wl.as_bits(w1), DEV))
        codec.init_caches(wa[-1])
    outs = [[torch.empty_like(c.weights_out) for c in layers] for _ in range(8)]
    pipe = runtime.LayerPipeline(layers)
    torch.cuda.synchronize()
    for i in range(8):
        pipe.step(wb if i % 2 == 0 else wa, outs[i])
    pipe.wait()
    torch.cuda.synchronize()
    for c in layers:
        c.check_status()
    for i in range(8):
        want = wb if i % 2 == 0 else wa
        for l in range(n_layers):
            assert torch.equal(outs[i][l][: want[l].numel()], want[l]), f"iteration {i}, layer {l}"


@pytest.mark.parametrize("dtype,block", [(0, 512), (1, 512), (0, 64)])
def test_full_size_layer_sampled_units(rt, dtype, block):
    """One full OLMoE-shaped layer (64 experts x 3 matrices, 16 shards: 3072 units, 402 653 184 values) in the
    launch configuration the benchmark times, generated on the device.  The round trip is checked everywhere
    (device-side comparison); messages, lengths, counts and caches of sampled units are checked against the
    oracle, which gets the units' weights before and after the step."""
    ciera, runtime = rt
    from oracle import ciera_oracle as ora

    name = NAME[dtype]
    vb = wl.VALUE_BYTES[name]
    shapes = [r * c for r, c in wl.olmoe_layer_shapes(64)]
    codec = runtime.LayerCodec.from_tensors(shapes, 16, name, block, DEV)
    n = codec.weights_bytes // vb
    gen = wl.make_generator(2024 + dtype, DEV)
    w0 = wl.init_weights(n, name, gen)
    w1 = wl.step_clustered(w0, gen, f=0.22)
    w2 = wl.step_adam_like(w1, gen)  # second step: every block changes
    b0, b1, b2 = (w.view(torch.uint8) for w in (w0, w1, w2))
    codec.init_caches(b0)
    rng = np.random.default_rng(5)
    picks = sorted(set(rng.integers(0, len(codec.units), 80).tolist()) | {0, len(codec.units) - 1})
    assert len(picks) >= 64
    wdt = WDT[dtype]
    prev = b0
    for cur in (b1, b2):
        codec.step(cur)
        torch.cuda.synchronize()
        codec.check_status()
        assert torch.equal(codec.weights_out[: cur.numel()], cur), "round trip is not bit-exact"
        assert torch.equal(codec.sender_cache, codec.receiver_cache)
        for ui in picks:
            u = codec.units[ui]
            lo, nn, mo, co = int(u["weights_off"]), int(u["n_values"]), int(u["msg_off"]), int(u["cache_off"])
            wp = prev[lo : lo + nn * vb].cpu().numpy().view(wdt)
            wc = cur[lo : lo + nn * vb].cpu().numpy().view(wdt)
            cache = ora.cache_init(wp, nn, dtype)
            m, wbytes, pay, cb = ora.encode(wc, cache, dtype, block)
            assert int(codec.wire_bytes[ui].item()) == wbytes and int(codec.changed_blocks[ui].item()) == cb
            assert np.array_equal(codec.msg_send[mo : mo + wbytes].cpu().numpy(), m), f"message of unit {ui}"
            assert np.array_equal(codec.msg_recv[mo : mo + wbytes].cpu().numpy(), m), f"transported message {ui}"
            assert np.array_equal(codec.sender_cache[co : co + nn].cpu().numpy(), cache)
        prev = cur
    q = int(codec.changed_blocks.sum().item()) / codec.n_blocks()
    assert q > (0.99 if block >= 256 else 0.8)  # the i.i.d. step changes (nearly) every block


@pytest.mark.parametrize("n_shards", [8, 64])
def test_config5_full_size_mixed_shapes(rt, n_shards):
    """The mixed-shape sweep at full size in ONE plan: 256 fine-grained experts x (2048x512, 2048x512, 512x2048)
    plus dense tensors of 4 KB ... 256 MB (bf16) and one ragged 1000-value tensor, cut into 8 or 64 shards.  At 8
    shards the 256 MB tensor gives units of 16.8 M values = 2048 tiles (tiles spread over the thread blocks,
    look-back between them, cooperative launch, per-tile counts from the prefix kernel at decode time); at 64
    shards the 4 KB tensor gives units of 32 values, far below the block size, and the ragged tensor a short-tail
    unit and an empty one.  Exponent changes are injected at 0.1 %, 1 %, 10 % and 50 %, value by value and in
    512-aligned segments, on the device.  After every step: the round trip is exact over the whole buffer (the
    gaps between units hold guard bytes on both sides of the comparison), both caches agree, and messages,
    lengths, counts and caches of sampled units equal the oracle's -- among them the first, a middle and the last
    shard of the 256 MB tensor, a 32-value unit, the short-tail unit and the empty unit."""
    ciera, runtime = rt
    from oracle import ciera_oracle as ora

    block = 512
    dense = wl.dense_tensor_sizes()
    sizes = [r * c for r, c in wl.fine_grained_layer_shapes(256)] + dense + [1000]
    codec = guard(runtime.LayerCodec.from_tensors(sizes, n_shards, "bf16", block, DEV, slack=256))
    units = codec.units
    n = codec.weights_bytes // 2
    first_of = lambda tensor: tensor * n_shards  # index of a tensor's first unit
    big, small, ragged = first_of(256 * 3 + len(dense) - 1), first_of(256 * 3), first_of(256 * 3 + len(dense))
    assert int(units[big]["n_values"]) == dense[-1] // n_shards
    special = [big, big + n_shards // 2, big + n_shards - 1, small, small + n_shards - 1]
    tail = [ragged + i for i in range(n_shards) if int(units[ragged + i]["n_values"]) < -(-1000 // n_shards)]
    assert any(int(units[i]["n_values"]) == 0 for i in tail) or n_shards == 8
    special += tail[:3]
    rng = np.random.default_rng(77 + n_shards)
    picks = sorted(set(special) | set(rng.integers(0, len(units), 16).tolist()))
    if n_shards == 8:
        assert codec.plan.n_tiles > 0 and int(units[big]["n_values"]) // 8192 == 2048
    else:
        assert int(units[small]["n_values"]) == 32

    gen = wl.make_generator(5005 + n_shards, DEV)
    w = wl.init_weights(n, "bf16", gen)
    gaps = codec.canaries.guards["weights_out"]
    gaps = gaps[gaps < w.numel() * 2]

    def as_bytes(t):
        b = t.view(torch.uint8)
        b[gaps] = codec.canaries.PATTERN  # not part of any unit: make both sides of the comparison agree there
        return b

    prev = as_bytes(w)
    codec.init_caches(prev)
    for c, seg in [(0.001, 0), (0.01, 0), (0.1, 0), (0.5, 0), (0.001, 512), (0.01, 512), (0.1, 512), (0.5, 512)]:
        w = wl.inject_exponent_changes(w, gen, c, seg)
        cur = as_bytes(w)
        codec.step(cur)
        torch.cuda.synchronize()
        codec.check_status()
        label = f"config5 shards={n_shards} c={c} seg={seg}"
        codec.canaries.check(label)
        assert torch.equal(codec.weights_out[: cur.numel()], cur), f"{label}: round trip is not bit-exact"
        assert torch.equal(codec.sender_cache, codec.receiver_cache), f"{label}: the two caches differ"
        for ui in picks:
            u = units[ui]
            lo, nn, mo, co = int(u["weights_off"]), int(u["n_values"]), int(u["msg_off"]), int(u["cache_off"])
            wp = prev[lo : lo + nn * 2].cpu().numpy().view(np.uint16)
            wc = cur[lo : lo + nn * 2].cpu().numpy().view(np.uint16)
            cache = ora.cache_init(wp, nn, 0)
            m, wbytes, pay, cb = ora.encode(wc, cache, 0, block)
            assert int(codec.wire_bytes[ui].item()) == wbytes, f"{label}: length of unit {ui} (N={nn})"
            assert int(codec.changed_blocks[ui].item()) == cb, f"{label}: changed blocks of unit {ui} (N={nn})"
            assert np.array_equal(codec.msg_send[mo : mo + wbytes].cpu().numpy(), m), f"{label}: message of unit {ui}"
            assert np.array_equal(codec.msg_recv[mo : mo + wbytes].cpu().numpy(), m), f"{label}: transported {ui}"
            assert np.array_equal(codec.sender_cache[co : co + nn].cpu().numpy(), cache), f"{label}: cache of {ui}"
        q = int(codec.changed_blocks.sum().item()) / codec.n_blocks()
        assert 0 < q <= 1
        prev = cur


@pytest.mark.parametrize("block", [512, 1])
def test_buffers_beyond_four_gib(rt, block):
    """(With blocks of 512 values, and of one value: the fine-block kernels and their prefix kernel.)
    One plan whose buffers are larger than 4 GiB each: 4.56 G bf16 values (9.1 GB of weights, 4.6 GB per cache,
    9.1 GB per message buffer), so that byte offsets pass 2^32 in every buffer and 2^33 in weights and messages --
    no 32-bit offset arithmetic survives this.  34 tensors of 128 Mi values in 4 shards (units of 4096 tiles: spread
    tiles, look-back, cooperative launch, prefix kernel) between short units at the start and, beyond all the
    marks, at the end.  Generated on the device in chunks.  After each of two steps (clustered, then 0.1 % of the
    exponents changed in segments) the round trip is exact over the whole buffer, both caches agree, the guard
    bytes are intact, and the units that straddle the 2^32 and 2^33 marks of each buffer, the first and the last
    units equal the oracle's messages, lengths, counts and caches."""
    ciera, runtime = rt
    from oracle import ciera_oracle as ora

    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 90e9:
        pytest.skip("needs 90 GB of free device memory")
    n_shards, big = 4, 1 << 27
    sizes = [1_000_001] + [big] * 34 + [1_000_001, 300_000, 4096 + 5]
    codec = guard(runtime.LayerCodec.from_tensors(sizes, n_shards, "bf16", block, DEV, slack=256))
    units = codec.units
    n = codec.weights_bytes // 2
    assert codec.weights_bytes > 2 ** 33 and codec.cache_bytes > 2 ** 32 and codec.msg_bytes > 2 ** 33

    def straddlers(off_key, length_of, marks):
        out = []
        for i, u in enumerate(units):
            lo = int(u[off_key])
            hi = lo + length_of(u)
            out += [i for m in marks if lo < m <= hi or (lo <= m < hi)]
        return out

    picks = set(straddlers("weights_off", lambda u: 2 * int(u["n_values"]), (2 ** 32, 2 ** 33)))
    picks |= set(straddlers("cache_off", lambda u: int(u["n_values"]), (2 ** 32,)))
    picks |= set(straddlers("msg_off", lambda u: int(u["msg_capacity"]), (2 ** 32, 2 ** 33)))
    assert len(picks) >= 2
    picks |= {i + d for i in picks for d in (-1, 1)}  # and their neighbours, which lie wholly beyond a mark
    picks |= {0, 1, len(units) // 2} | set(range(len(units) - 3 * n_shards, len(units)))
    picks = sorted(picks)
    assert int(units[picks[-1]]["weights_off"]) > 2 ** 33 and int(units[picks[-1]]["cache_off"]) > 2 ** 32

    gen = wl.make_generator(4242, DEV)
    chunk = 1 << 28

    def chunked(make, like=None):
        out = torch.empty(n, dtype=torch.bfloat16, device=DEV)
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            out[lo:hi] = make(hi - lo) if like is None else make(like[lo:hi])
        return out

    gaps = codec.canaries.guards["weights_out"]
    gaps = gaps[gaps < 2 * n]

    def as_bytes(t):
        b = t.view(torch.uint8)
        b[gaps] = codec.canaries.PATTERN  # not part of any unit: make both sides of the comparison agree there
        return b

    w = chunked(lambda m: wl.init_weights(m, "bf16", gen))
    prev = as_bytes(w)
    codec.init_caches(prev)
    steps = [lambda x: wl.step_clustered(x, gen, f=0.22), lambda x: wl.inject_exponent_changes(x, gen, 0.001, 512)]
    for t, make in enumerate(steps):
        w_next = chunked(make, like=w)
        cur = as_bytes(w_next)
        codec.step(cur)
        torch.cuda.synchronize()
        codec.check_status()
        label = f"beyond 4 GiB, step {t}"
        codec.canaries.check(label)
        assert torch.equal(codec.weights_out[: cur.numel()], cur), f"{label}: round trip is not bit-exact"
        assert torch.equal(codec.sender_cache, codec.receiver_cache), f"{label}: the two caches differ"
        for ui in picks:
            u = units[ui]
            lo, nn, mo, co = int(u["weights_off"]), int(u["n_values"]), int(u["msg_off"]), int(u["cache_off"])
            wp = prev[lo : lo + nn * 2].cpu().numpy().view(np.uint16)
            wc = cur[lo : lo + nn * 2].cpu().numpy().view(np.uint16)
            cache = ora.cache_init(wp, nn, 0)
            m, wbytes, pay, cb = ora.encode(wc, cache, 0, block)
            assert int(codec.wire_bytes[ui].item()) == wbytes, f"{label}: length of unit {ui} (N={nn})"
            assert int(codec.changed_blocks[ui].item()) == cb, f"{label}: changed blocks of unit {ui} (N={nn})"
            assert np.array_equal(codec.msg_send[mo : mo + wbytes].cpu().numpy(), m), f"{label}: message of unit {ui}"
            assert np.array_equal(codec.msg_recv[mo : mo + wbytes].cpu().numpy(), m), f"{label}: transported {ui}"
            assert np.array_equal(codec.sender_cache[co : co + nn].cpu().numpy(), cache), f"{label}: cache of {ui}"
        q = int(codec.changed_blocks.sum().item()) / codec.n_blocks()
        assert 0 < q < 0.5
        del prev
        w, prev = w_next, cur
    if block < 16:  # the hashed sender takes blocks of 16 values and more
        return

    # a third step through the hashed sender (its messages are the exact sender's) and the entropy stage, whose
    # scratch (one slot per 4096 values) is larger than 4 GiB here as well
    from oracle import rans_oracle as rans

    codec.init_hash_cache(prev)
    cur = as_bytes(chunked(lambda x: wl.step_clustered(x, gen, f=0.22), like=w))
    codec.encode_hashed(cur)
    torch.cuda.synchronize()
    hashed_wire, hashed_changed = codec.wire_bytes.clone(), codec.changed_blocks.clone()
    hashed_msgs = {ui: codec.msg_send[int(units[ui]["msg_off"]) : int(units[ui]["msg_off"]) + int(hashed_wire[ui].item())].clone()
                   for ui in picks}
    codec.msg_send.zero_()
    guard(codec)  # (the fill went over the guard bytes between the slots: arm them again)
    codec.encode(cur)
    torch.cuda.synchronize()
    assert torch.equal(codec.wire_bytes, hashed_wire) and torch.equal(codec.changed_blocks, hashed_changed)
    raw_msgs = {}
    for ui in picks:
        mo = int(units[ui]["msg_off"])
        raw_msgs[ui] = codec.msg_send[mo : mo + int(hashed_wire[ui].item())].cpu().numpy()
        assert np.array_equal(raw_msgs[ui], hashed_msgs[ui].cpu().numpy()), f"hashed sender, unit {ui}"
    assert codec.plan.entropy_scratch_bytes > 2 ** 32
    codec.entropy_encode()
    torch.cuda.synchronize()
    for ui in picks:
        u = units[ui]
        want = rans.entropy_encode_message(raw_msgs[ui], int(u["n_values"]), 0, block)
        assert int(codec.wire_bytes[ui].item()) == want.size, f"coded length of unit {ui}"
        mo = int(u["msg_off"])
        assert np.array_equal(codec.msg_send[mo : mo + want.size].cpu().numpy(), want), f"coded message of unit {ui}"
    assert int(codec.wire_bytes.sum().item()) < int(hashed_wire.sum().item())
    codec.transport()
    codec.entropy_decode()
    codec.decode()
    torch.cuda.synchronize()
    codec.check_status()
    codec.canaries.check("beyond 4 GiB, hashed sender and entropy stage")
    assert torch.equal(codec.wire_bytes, hashed_wire)
    assert torch.equal(codec.weights_out[: cur.numel()], cur), "round trip through the entropy stage is not bit-exact"
    assert torch.equal(codec.sender_cache, codec.receiver_cache)


def test_one_unit_of_more_than_two_to_the_32_values(rt):
    """A single unit of 2^32 + 24 581 bf16 values (8.6 GB; 524 292 tiles, a short last block of 5 values): offsets
    INSIDE the unit pass 2^32 in the sign-plus-mantissa section, in the payload (the look-back carries byte counts
    beyond 32 bits) and in the caches.  The CPU oracle would need tens of GB of host memory for this, so the
    message is checked on the device against the definition written with plain torch operations, chunk by
    chunk: block flags = "some exponent of the block differs", bitmap = the flags LSB-first, sign-plus-mantissa
    of every value, payload = the exponents of the flagged blocks in order, length and count, caches = the new
    exponents, output = the input."""
    ciera, runtime = rt
    from oracle import ciera_oracle as ora

    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 90e9:
        pytest.skip("needs 90 GB of free device memory")
    block, n = 512, 2 ** 32 + 3 * 8192 + 5
    codec = guard(runtime.LayerCodec.from_tensors([n], 1, "bf16", block, DEV, slack=256))
    assert len(codec.units) == 1 and int(codec.units[0]["n_values"]) == n
    nb = -(-n // block)
    pay_off = ora.payload_offset(n, 0, block)
    sm_off = pay_off - (n + 15) // 16 * 16
    assert sm_off == (-(-nb // 8) + 15) // 16 * 16
    gen = wl.make_generator(99, DEV)
    chunk = 1 << 28  # a multiple of the block size and of 8 blocks
    w0 = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    w1 = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        w0[lo:hi] = wl.init_weights(hi - lo, "bf16", gen)
        w1[lo:hi] = wl.step_clustered(w0[lo:hi], gen, f=0.22)
    b0, b1 = w0.view(torch.uint8), w1.view(torch.uint8)
    codec.init_caches(b0)
    codec.step(b1)
    torch.cuda.synchronize()
    codec.check_status()
    codec.canaries.check("one unit of more than 2^32 values")
    assert torch.equal(codec.weights_out[: 2 * n], b1), "round trip is not bit-exact"

    def exponents(w):  # bf16: bits 14..7
        return ((w.view(torch.int16).to(torch.int32) >> 7) & 0xFF).to(torch.uint8)

    def sign_mantissa(w):  # sign << 7 | mantissa
        v = w.view(torch.int16).to(torch.int32)
        return (((v >> 8) & 0x80) | (v & 0x7F)).to(torch.uint8)

    msg = codec.msg_send
    bit_weights = torch.tensor([1, 2, 4, 8, 16, 32, 64, 128], dtype=torch.int32, device=DEV)
    sent = changed = 0
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        e0, e1 = exponents(w0[lo:hi]), exponents(w1[lo:hi])
        assert torch.equal(codec.sender_cache[lo:hi], e1) and torch.equal(codec.receiver_cache[lo:hi], e1), f"caches at {lo}"
        assert torch.equal(msg[sm_off + lo : sm_off + hi], sign_mantissa(w1[lo:hi])), f"sign-plus-mantissa at {lo}"
        m = hi - lo
        diff = e0 != e1
        pad = (-m) % (8 * block)
        if pad:
            diff = torch.cat([diff, torch.zeros(pad, dtype=torch.bool, device=DEV)])
        flags = diff.view(-1, block).any(dim=1)  # a multiple of 8 flags
        want_bitmap = (flags.view(-1, 8).to(torch.int32) * bit_weights).sum(dim=1).to(torch.uint8)
        first_byte = lo // block // 8
        nbytes = -(-(-(-m // block)) // 8)
        assert torch.equal(msg[first_byte : first_byte + nbytes], want_bitmap[:nbytes]), f"bitmap at {lo}"
        mask = flags.repeat_interleave(block)[:m]
        want_payload = e1[mask]
        assert torch.equal(msg[pay_off + sent : pay_off + sent + want_payload.numel()], want_payload), f"payload at {lo}"
        sent += int(want_payload.numel())
        changed += int(flags.sum().item())
    assert sent > 2 ** 30 // 2 and int(codec.changed_blocks[0].item()) == changed
    assert int(codec.wire_bytes[0].item()) == pay_off + sent
    assert pay_off > 2 ** 32 and torch.equal(codec.msg_recv[: pay_off + sent], msg[: pay_off + sent])

    # the same step by the hashed sender gives the same message; then once through the entropy stage and back
    # (its chain of launches for long units, a quarter of a million segments)
    del e0, e1, diff, flags, mask, want_payload, want_bitmap
    codec.init_caches(b0)
    codec.init_hash_cache(b0)
    # (the hashed call writes into msg_send: keep the exact message in msg_recv's place)
    codec.msg_recv[: pay_off + sent].copy_(msg[: pay_off + sent])
    msg.zero_()
    guard(codec)
    codec.encode_hashed(b1)
    torch.cuda.synchronize()
    codec.check_status()
    assert int(codec.wire_bytes[0].item()) == pay_off + sent and int(codec.changed_blocks[0].item()) == changed
    assert torch.equal(msg[: pay_off + sent], codec.msg_recv[: pay_off + sent]), "hashed sender's message differs"
    codec.encode(b1)
    codec.entropy_encode()
    torch.cuda.synchronize()
    coded = int(codec.wire_bytes[0].item())
    assert pay_off < coded < pay_off + sent * 6 // 10  # exponents of Gaussian weights: well under 5 bits each
    codec.transport()
    codec.entropy_decode()
    codec.decode()
    torch.cuda.synchronize()
    codec.check_status()
    codec.canaries.check("one unit of more than 2^32 values, entropy stage")
    assert int(codec.wire_bytes[0].item()) == pay_off + sent
    assert torch.equal(codec.weights_out[: 2 * n], b1), "round trip through the entropy stage is not bit-exact"
    assert torch.equal(codec.sender_cache[:n], codec.receiver_cache[:n])


@pytest.mark.parametrize("sizes", [[], [0], [0, 0, 0]])
@pytest.mark.parametrize("dtype_name", ["bf16", "fp32", "fp16"])
def test_tables_without_values_run_through_every_entry_point(rt, sizes, dtype_name):
    """No units, or only units without values: every call returns without touching anything."""
    ciera, runtime = rt
    codec = runtime.LayerCodec.from_tensors(sizes, 1, dtype_name, 64, DEV)
    w = torch.zeros(16, dtype=torch.uint8, device=DEV)
    codec.init_caches(None)
    codec.init_caches(w)
    launches0 = ciera.kernel_launch_count()
    codec.step(w)
    ciera.encode_noalloc(codec.plan, w, codec.sender_cache, codec.msg_send, codec.wire_bytes, codec.changed_blocks,
                         codec.status)
    if dtype_name != "fp16":
        codec.init_hash_cache(None)
        codec.encode_hashed(w)
        codec.entropy_encode()
        codec.entropy_decode()
    host_in = torch.zeros(16, dtype=torch.uint8).pin_memory()
    host_out = torch.zeros(16, dtype=torch.uint8).pin_memory()
    wire_host = torch.zeros(max(len(codec.units), 1), dtype=torch.int64).pin_memory()
    codec.step_host(host_in, host_out, w, wire_host)
    torch.cuda.synchronize()
    codec.check_status()
    assert int(codec.wire_bytes.sum().item()) == 0 and int(codec.changed_blocks.sum().item()) == 0
    assert ciera.kernel_launch_count() - launches0 == 0


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block", [1, 64, 512])
def test_tightly_packed_layout_in_shuffled_order(rt, dtype, block):
    """Buffers laid out with the minimum alignment (16 bytes) and the units of the table listed in a
    shuffled order: every offset the kernels derive must hold without the 256-byte padding of the
    other tests."""
    ciera, runtime = rt
    sizes = [8192 * 2 + 24, 100, 70_001, 8, 40_000, 8192, 12_345, 0, 131_072]
    code = dtype
    units, wb, cb, mb = wl.layout_units(sizes, 1, 2 if dtype == 0 else 4,
                                        lambda n: ciera.message_capacity(n, code, block), align=16)
    rng = np.random.default_rng(12 + block)
    units = units[rng.permutation(len(units))]
    codec = guard(runtime.LayerCodec(units, NAME[dtype], block, wb, cb, mb, DEV, slack=256))
    assert codec.canaries.guarded_bytes() > 5 * 256  # the slack and the 16-byte alignment gaps
    table = OracleTable(codec.units, dtype, block, codec.cache_bytes, codec.msg_bytes)
    n = wb // (2 if dtype == 0 else 4)
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 90 + block, 2, "adam")]
    _run_trajectory(rt, codec, table, traj, dtype, label=f"tight-{NAME[dtype]}-B{block}")
    _run_trajectory(rt, codec, table, traj[:2], dtype, zero_cache=True, label=f"tight-zero-{NAME[dtype]}-B{block}")


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block,rate", [(16, 0.9), (64, 0.9), (128, 0.95), (256, 0.5), (512, 0.5), (512, 0.06),
                                        (4096, 0.5)])
def test_scattered_unchanged_blocks(rt, dtype, block, rate):
    """Whole blocks change at a given rate, the unchanged ones scattered between them: the receiver
    fetches the cached exponents of unchanged blocks as a span, run by run, or piece by piece
    depending on how many there are and how they lie."""
    codec, table, n = _make(rt, [600_000, 131_072, 70_001], 2, dtype, block)
    gen = wl.make_generator(4100 + block)
    w0 = wl.init_weights(n, NAME[dtype], gen)
    w1 = wl.inject_exponent_changes(w0, gen, rate, seg=block)
    w2 = wl.inject_exponent_changes(w1, gen, rate, seg=block)
    stats = _run_trajectory(rt, codec, table, [wl.as_bits(w) for w in (w0, w1, w2)], dtype,
                            label=f"scattered-{NAME[dtype]}-B{block}-{rate}")
    changed, blocks = stats[-1]
    assert 0 < changed < blocks  # (segments are aligned in the buffer, not in every unit: the rate is only roughly `rate`)
