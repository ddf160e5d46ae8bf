"""Test-side runners: the CPU oracle over a whole unit table, and comparison with the CUDA path.

Lives in tests/ and is used by tests only.  The oracle runner keeps its own flat caches in the
same layout as the device buffers so that results can be compared byte for byte."""
import numpy as np
import torch

from oracle import ciera_oracle as ora

VB = {0: 2, 1: 4, 2: 2}
WDT = {0: np.uint16, 1: np.uint32, 2: np.uint16}


class OracleTable:
    def __init__(self, units, dtype, block, cache_bytes, msg_bytes):
        self.units, self.dtype, self.block = units, dtype, block
        self.cache_s = np.zeros(max(cache_bytes, 16), np.uint8)
        self.cache_r = np.zeros(max(cache_bytes, 16), np.uint8)
        self.msg_bytes = msg_bytes

    def _w(self, w_flat, u):
        lo = int(u["weights_off"]) // VB[self.dtype]
        return w_flat[lo : lo + int(u["n_values"])]

    def init_caches(self, w_flat):
        for u in self.units:
            n, co = int(u["n_values"]), int(u["cache_off"])
            c = ora.cache_init(None if w_flat is None else self._w(w_flat, u), n, self.dtype)
            self.cache_s[co : co + n] = c
            self.cache_r[co : co + n] = c

    def step(self, w_flat):
        """Encode + decode every unit.  Returns dict with flat message buffer (only the first
        wire[u] bytes of each slot are meaningful), wire, changed, payload, recon."""
        nu = len(self.units)
        msgs = np.zeros(max(self.msg_bytes, 16), np.uint8)
        wire = np.zeros(nu, np.uint64)
        chg = np.zeros(nu, np.uint32)
        pay = np.zeros(nu, np.uint64)
        recon = np.zeros_like(w_flat)
        for i, u in enumerate(self.units):
            n, co, mo = int(u["n_values"]), int(u["cache_off"]), int(u["msg_off"])
            cs = self.cache_s[co : co + n].copy()
            m, wb, pb, cb = ora.encode(self._w(w_flat, u), cs, self.dtype, self.block)
            self.cache_s[co : co + n] = cs
            msgs[mo : mo + wb] = m
            wire[i], chg[i], pay[i] = wb, cb, pb
            cr = self.cache_r[co : co + n].copy()
            out = ora.decode(m, cr, self.dtype, self.block)
            self.cache_r[co : co + n] = cr
            lo = int(u["weights_off"]) // VB[self.dtype]
            recon[lo : lo + n] = out
        return dict(msgs=msgs, wire=wire, chg=chg, pay=pay, recon=recon)


class Canaries:
    """Guard bytes around everything a step may write (the memory checker of the CUDA toolkit is not
    available on the test machines).  The gaps that the layout leaves between the units inside
    ``weights_out``, both caches and both message buffers, the ``slack`` bytes behind each of those
    buffers, and the slack entries behind the per-unit outputs are filled with a pattern when the
    object is made; ``check`` asserts that every one of them is untouched.  No kernel has any business
    there: a store that lands in a gap corrupts a neighbouring tensor in a real run without showing up
    in any comparison of the units' own bytes.  (Inside a message slot the bytes between the reported
    length and the slot's capacity are unspecified, so only the bytes past the capacity are guarded.)"""

    PATTERN = 0xA5

    def __init__(self, codec):
        self.codec = codec
        vb = VB[codec.dtype]
        u = codec.units
        n = u["n_values"].astype(np.int64)
        spans = {
            "weights_out": (u["weights_off"].astype(np.int64), n * vb),
            "sender_cache": (u["cache_off"].astype(np.int64), n),
            "receiver_cache": (u["cache_off"].astype(np.int64), n),
            "msg_send": (u["msg_off"].astype(np.int64), u["msg_capacity"].astype(np.int64)),
            "msg_recv": (u["msg_off"].astype(np.int64), u["msg_capacity"].astype(np.int64)),
        }
        self.guards = {}
        for name, (off, length) in spans.items():
            full = codec.allocations.get(name)
            if full is None:
                continue
            idx = torch.from_numpy(self._uncovered(off, length, full.numel())).to(full.device)
            full[idx] = self.PATTERN
            self.guards[name] = idx
        self.tails = {}
        for name, live in (("wire_bytes", len(u)), ("changed_blocks", len(u))):
            full = codec.allocations[name]
            live = max(live, 1)
            full[live:] = 0x5A5A5A5A
            self.tails[name] = live

    @staticmethod
    def _uncovered(off, length, total):
        """Indices of [0, total) that lie in no [off_i, off_i + length_i)."""
        keep = length > 0
        off, length = off[keep], length[keep]
        order = np.argsort(off, kind="stable")
        off, end = off[order], (off + length)[order]
        starts = np.concatenate([[0], end])
        stops = np.concatenate([off, [total]])
        assert np.all(stops >= starts), "units overlap"
        parts = [np.arange(a, b, dtype=np.int64) for a, b in zip(starts, stops) if b > a]
        return np.concatenate(parts) if parts else np.zeros(0, np.int64)

    def guarded_bytes(self):
        return sum(int(i.numel()) for i in self.guards.values())

    def check(self, label=""):
        for name, idx in self.guards.items():
            full = self.codec.allocations[name]
            bad = (full[idx] != self.PATTERN).nonzero()
            assert bad.numel() == 0, (f"{label}: a store landed outside the units' bytes of {name}, first at byte "
                                      f"{int(idx[bad[0, 0]])} of the buffer")
        for name, live in self.tails.items():
            full = self.codec.allocations[name]
            assert bool((full[live:] == 0x5A5A5A5A).all()), f"{label}: entries past the last unit of {name} were written"


def guard(codec):
    """Arms the guard bytes of a codec made with ``slack`` > 0 (see Canaries); returns the codec."""
    codec.canaries = Canaries(codec)
    return codec


def to_dev_bytes(bits: np.ndarray, device) -> torch.Tensor:
    """Raw bytes of a host bit-pattern array, on the device (padded to >= 16 bytes)."""
    b = np.ascontiguousarray(bits).view(np.uint8)
    if b.size < 16:
        b = np.concatenate([b, np.zeros(16 - b.size, np.uint8)])
    return torch.from_numpy(b.copy()).to(device)


def dev_to_bits(t: torch.Tensor, dtype: int, n: int) -> np.ndarray:
    return t.cpu().numpy().view(WDT[dtype])[:n]


def compare_step(codec, exp, w_flat, label=""):
    """Bit-exact comparison of one finished GPU step (codec: LayerCodec) with the oracle's."""
    units = codec.units
    nu = len(units)
    wire = codec.wire_bytes.cpu().numpy().astype(np.uint64)[:nu]
    chg = codec.changed_blocks.cpu().numpy().astype(np.uint32)[:nu]
    assert np.array_equal(wire, exp["wire"]), f"{label}: wire bytes differ"
    assert np.array_equal(chg, exp["chg"]), f"{label}: changed-block counts differ"
    ms = codec.msg_send.cpu().numpy()
    mr = codec.msg_recv.cpu().numpy()
    for i, u in enumerate(units):
        mo, wb = int(u["msg_off"]), int(wire[i])
        if not np.array_equal(ms[mo : mo + wb], exp["msgs"][mo : mo + wb]):
            bad = np.nonzero(ms[mo : mo + wb] != exp["msgs"][mo : mo + wb])[0]
            raise AssertionError(f"{label}: message of unit {i} (N={int(u['n_values'])}) differs at bytes {bad[:8]}")
        assert np.array_equal(mr[mo : mo + wb], exp["msgs"][mo : mo + wb]), f"{label}: transported message {i}"
    return wire, chg


def sender_scratch_is_clean(codec) -> bool:
    """The calls find their counters in the workspace (one status word per tile and 16 bytes of counters for the
    sender, then 16 bytes for transport and receiver) all zero and have to hand them back all zero: there is no
    clearing launch in front of any kernel."""
    n = 8 * codec.plan.n_tiles + 32
    clean = not bool(codec.workspace[:n].any().item())
    hw = getattr(codec, "hashed_workspace", None)
    if hw is not None:
        clean = clean and not bool(hw[:n].any().item())
    return clean


def compare_caches(codec, table, label=""):
    if getattr(codec, "canaries", None) is not None:
        codec.canaries.check(label)
    assert sender_scratch_is_clean(codec), f"{label}: the counters in the scratch were not handed back all zero"
    cs = codec.sender_cache.cpu().numpy()
    cr = codec.receiver_cache.cpu().numpy()
    for i, u in enumerate(codec.units):
        co, n = int(u["cache_off"]), int(u["n_values"])
        assert np.array_equal(cs[co : co + n], table.cache_s[co : co + n]), f"{label}: sender cache unit {i}"
        assert np.array_equal(cr[co : co + n], table.cache_r[co : co + n]), f"{label}: receiver cache unit {i}"


def compare_recon(codec, exp, w_flat, dtype, label=""):
    out = codec.weights_out.cpu().numpy().view(WDT[dtype])
    for i, u in enumerate(codec.units):
        lo, n = int(u["weights_off"]) // VB[dtype], int(u["n_values"])
        assert np.array_equal(out[lo : lo + n], exp["recon"][lo : lo + n]), f"{label}: reconstruction unit {i}"
        assert np.array_equal(out[lo : lo + n], w_flat[lo : lo + n]), f"{label}: round trip unit {i}"
