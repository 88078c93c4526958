"""Seeded synthetic inputs for non-uniform all-to-all exchanges.

This module only *generates inputs* (count matrices, displacement tables and
payload bytes).  It contains none of the exchange arithmetic: no radix digits,
no rounds, no prefix sums over slots.  Both the CPU oracle's tests and the CUDA
path's tests draw their inputs from here, so that the two are compared on the
very same bytes.

Every value is a pure function of ``(seed, stream, index)`` through one
counter-based 64-bit mixer (the splitmix64 finaliser applied to a Weyl
sequence), written with torch integer ops so that the same code runs on the
CPU and on a CUDA device.  Any single payload word can therefore be
regenerated on its own, which is what the full-size sampled parity checks do.

Workload shapes (the paper draws block sizes uniformly from [0, S] and also
reports a power-law case with rare large blocks and many empty ones; the five
shapes below follow those, plus a mixture-of-experts token dispatch):

* ``c1``  P=8,    int32 elements, counts U{0..64}; element value encodes
          (src, dst, idx) so a misplaced element names its true home.
* ``c2``  P=64,   bytes, counts uniform over {0,16,...,4096}.
* ``c3``  P=256,  float32 elements, finite Zipf(1.2) counts on [0, 8192].
* ``c4``  P=64,   8192 tokens per rank routed top-2 by Gaussian logits; a
          block is the chosen tokens' rows of ``hidden`` bf16 values.
* ``c5``  P=2048, bytes, 30 % of pairs empty, the rest U{0..512}.

plus the paper's other patterns at P=4096: ``normal`` and ``powerlaw`` block
sizes capped at 1024 bytes, and the two FFT transposes ``fft_n1`` / ``fft_n2``.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

_MASK63 = (1 << 63) - 1


def _i64(v: int) -> int:
    """Wrap an unsigned 64-bit constant into the signed range torch uses."""
    v &= (1 << 64) - 1
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _i64(0x9E3779B97F4A7C15)
_STREAM = _i64(0xD1B54A32D192ED03)
_SEEDK = _i64(0x8CB92BA72F3D8DD7)
_M1 = _i64(0xBF58476D1CE4E5B9)
_M2 = _i64(0x94D049BB133111EB)

# stream ids
S_COUNTS = 1
S_PAYLOAD = 2
S_ZERO = 3
S_GAPS = 4
S_LOGITS = 5
S_BIAS = 6


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def mix64(seed: int, stream: int, index: torch.Tensor) -> torch.Tensor:
    """64 pseudo-random bits per index; a pure function of its arguments.

    ``index`` is an int64 tensor (any device); the result has the same shape
    and device, and holds the 64 bits in two's complement.
    """
    base = _i64(seed * 0x8CB92BA72F3D8DD7 + stream * 0xD1B54A32D192ED03)
    z = index * _GOLDEN + base
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def uniform_int(seed: int, stream: int, n: int, lo: int, hi: int,
                device="cpu") -> torch.Tensor:
    """n integers uniform on [lo, hi] (inclusive) as int64."""
    bits = _lsr(mix64(seed, stream, torch.arange(n, dtype=torch.int64, device=device)), 11)
    return lo + bits % (hi - lo + 1)


def uniform_unit(seed: int, stream: int, n: int, device="cpu") -> torch.Tensor:
    """n doubles uniform on [0, 1) with 53 random bits each."""
    bits = _lsr(mix64(seed, stream, torch.arange(n, dtype=torch.int64, device=device)), 11)
    return bits.to(torch.float64) * (1.0 / (1 << 53))


def payload_words(seed: int, first_word: int, n_words: int, device="cpu",
                  out: torch.Tensor | None = None) -> torch.Tensor:
    """Payload as little-endian 64-bit words ``first_word .. first_word+n-1``."""
    idx = torch.arange(first_word, first_word + n_words, dtype=torch.int64, device=device)
    w = mix64(seed, S_PAYLOAD, idx)
    if out is not None:
        out.copy_(w)
        return out
    return w


def payload_bytes(seed: int, n_bytes: int, device="cpu", chunk_words: int = 1 << 26
                  ) -> torch.Tensor:
    """``n_bytes`` payload bytes: byte ``b`` is byte ``b % 8`` of word ``b // 8``."""
    n_words = (n_bytes + 7) // 8
    buf = torch.empty(max(n_words, 1), dtype=torch.int64, device=device)
    for w0 in range(0, n_words, chunk_words):
        w1 = min(n_words, w0 + chunk_words)
        payload_words(seed, w0, w1 - w0, device=device, out=buf[w0:w1])
    return buf.view(torch.uint8)[:n_bytes]


def payload_byte_at(seed: int, byte_index: torch.Tensor) -> torch.Tensor:
    """The payload byte at each global byte index (int64 tensor) as uint8."""
    w = mix64(seed, S_PAYLOAD, byte_index >> 3)
    return ((w >> ((byte_index & 7) * 8)) & 0xFF).to(torch.uint8)


@dataclasses.dataclass
class Workload:
    """One all-to-all problem over ``P`` ranks held in single send/recv buffers.

    Counts and displacements are in elements of ``elem_size`` bytes.
    ``sendcounts[s, d]`` elements go from rank s to rank d; rank p's send
    region starts ``sendbase[p]`` elements into the send buffer and block
    (p -> d) sits ``sdispls[p, d]`` elements into that region; likewise
    ``recvbase`` / ``rdispls[d, s]`` on the receiving side.
    """
    name: str
    P: int
    elem_size: int
    seed: int
    sendcounts: np.ndarray      # (P, P) int64
    sdispls: np.ndarray         # (P, P) int64
    rdispls: np.ndarray         # (P, P) int64
    sendbase: np.ndarray        # (P,) int64
    recvbase: np.ndarray        # (P,) int64
    send_elems: int             # extent of the send buffer, elements
    recv_elems: int             # extent of the recv buffer, elements
    radices: tuple = ()
    hier: tuple | None = None   # (l, g)
    hier_radices: tuple = ()    # ((rl, rg), ...)
    payload_kind: str = "bytes"  # "bytes" | "tagged_int32"

    @property
    def recvcounts(self) -> np.ndarray:
        return np.ascontiguousarray(self.sendcounts.T)

    @property
    def payload_bytes_total(self) -> int:
        return int(self.sendcounts.sum()) * self.elem_size

    @property
    def send_bytes(self) -> int:
        return self.send_elems * self.elem_size

    @property
    def recv_bytes(self) -> int:
        return self.recv_elems * self.elem_size

    def make_send(self, device="cpu") -> torch.Tensor:
        """The send buffer as a uint8 tensor of ``send_bytes`` bytes."""
        if self.payload_kind == "tagged_int32":
            assert self.elem_size == 4
            buf = np.full(self.send_elems, -1, dtype=np.int32)
            for s in range(self.P):
                for d in range(self.P):
                    c = int(self.sendcounts[s, d])
                    o = int(self.sendbase[s] + self.sdispls[s, d])
                    buf[o:o + c] = (s << 20) | (d << 10) | np.arange(c, dtype=np.int32)
            return torch.from_numpy(buf).view(torch.uint8).to(device)
        return payload_bytes(self.seed, self.send_bytes, device=device)

    def make_recv(self, device="cpu", fill: int = 0xA5) -> torch.Tensor:
        """A receive buffer pre-filled with a canary byte."""
        return torch.full((max(self.recv_bytes, 1),), fill, dtype=torch.uint8,
                          device=device)[:self.recv_bytes]


def _finish(name, P, elem_size, seed, counts, gaps=False, **kw) -> Workload:
    """Lay blocks out back to back (or with seeded gaps) in both buffers."""
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    recvc = counts.T
    if gaps:
        gs = uniform_int(seed, S_GAPS, P * P, 0, 3).numpy().reshape(P, P)
        gr = uniform_int(seed, S_GAPS, 2 * P * P, 0, 3).numpy()[P * P:].reshape(P, P)
    else:
        gs = np.zeros((P, P), dtype=np.int64)
        gr = np.zeros((P, P), dtype=np.int64)
    # block (p, j) starts after the earlier blocks of the row and their gaps
    ssz = counts + gs
    rsz = recvc + gr
    sd = np.cumsum(ssz, axis=1) - ssz + gs
    rd = np.cumsum(rsz, axis=1) - rsz + gr
    srow = ssz.sum(axis=1)
    rrow = rsz.sum(axis=1)
    sb = np.cumsum(srow) - srow
    rb = np.cumsum(rrow) - rrow
    return Workload(name=name, P=P, elem_size=elem_size, seed=seed, sendcounts=counts,
                    sdispls=np.ascontiguousarray(sd), rdispls=np.ascontiguousarray(rd),
                    sendbase=sb.astype(np.int64), recvbase=rb.astype(np.int64),
                    send_elems=int(srow.sum()), recv_elems=int(rrow.sum()), **kw)


def bench_seed(cfg: int) -> int:
    return 241102581 * 16 + cfg


def make_c1(seed: int | None = None, P: int = 8, gaps: bool = False) -> Workload:
    seed = bench_seed(1) if seed is None else seed
    c = uniform_int(seed, S_COUNTS, P * P, 0, 64).numpy().reshape(P, P)
    return _finish("c1", P, 4, seed, c, gaps=gaps, radices=(2,), payload_kind="tagged_int32")


def make_c2(seed: int | None = None, P: int = 64, max_bytes: int = 4096,
            gaps: bool = False) -> Workload:
    seed = bench_seed(2) if seed is None else seed
    c = 16 * uniform_int(seed, S_COUNTS, P * P, 0, max_bytes // 16).numpy().reshape(P, P)
    if gaps:  # keep every displacement a multiple of 16 bytes
        w = _finish("c2", P, 16, seed, c // 16, gaps=True)
        return dataclasses.replace(
            w, elem_size=1, sendcounts=w.sendcounts * 16, sdispls=w.sdispls * 16,
            rdispls=w.rdispls * 16, sendbase=w.sendbase * 16, recvbase=w.recvbase * 16,
            send_elems=w.send_elems * 16, recv_elems=w.recv_elems * 16,
            radices=(2, 4, 8, 16, 64))
    return _finish("c2", P, 1, seed, c, radices=(2, 4, 8, 16, 64))


def zipf_counts(seed: int, n: int, s: float = 1.2, cmax: int = 8192) -> np.ndarray:
    """n draws from Pr[c] proportional to (c+1)^-s on {0..cmax}, by inverse CDF."""
    pmf = (np.arange(cmax + 1, dtype=np.float64) + 1.0) ** (-s)
    cdf = np.cumsum(pmf)
    cdf /= cdf[-1]
    u = uniform_unit(seed, S_COUNTS, n).numpy()
    return np.minimum(np.searchsorted(cdf, u, side="right"), cmax).astype(np.int64)


def make_c3(seed: int | None = None, l: int = 16, g: int = 16, cmax: int = 8192,
            gaps: bool = False) -> Workload:
    seed = bench_seed(3) if seed is None else seed
    P = l * g
    c = zipf_counts(seed, P * P, 1.2, cmax).reshape(P, P)
    rr = tuple(r for r in (2, 4, 16))
    return _finish("c3", P, 4, seed, c, gaps=gaps, hier=(l, g),
                   hier_radices=tuple((a, b) for a in rr if a <= max(2, l)
                                      for b in rr if b <= max(2, g)))


def moe_top2_routing(seed: int, P: int, tokens: int, skew: bool = False):
    """(first, second): the two destinations of every token, arrays [P, tokens].

    Logits are i.i.d. N(0,1) by Box-Muller on the counter-based generator; the
    softmax is monotone, so the two largest logits are the top-2 experts; ties
    go to the lower index.  ``skew`` adds one N(0,1) bias per destination,
    shared by all ranks.
    """
    first = np.zeros((P, tokens), dtype=np.int64)
    second = np.zeros((P, tokens), dtype=np.int64)
    bias = None
    if skew:
        u1 = uniform_unit(seed, S_BIAS, 2 * P).numpy()
        bias = np.sqrt(-2.0 * np.log(1.0 - u1[:P])) * np.cos(2.0 * math.pi * u1[P:])
    per = tokens * P
    for s in range(P):
        idx = torch.arange(2 * s * per, 2 * (s + 1) * per, dtype=torch.int64)
        bits = _lsr(mix64(seed, S_LOGITS, idx), 11).to(torch.float64) * (1.0 / (1 << 53))
        u = bits.numpy().reshape(2, tokens, P)
        z = np.sqrt(-2.0 * np.log(1.0 - u[0])) * np.cos(2.0 * math.pi * u[1])
        if bias is not None:
            z = z + bias[None, :]
        first[s] = np.argmax(z, axis=1)
        z[np.arange(tokens), first[s]] = -np.inf
        second[s] = np.argmax(z, axis=1)
    return first, second


def moe_top2_counts(seed: int, P: int, tokens: int, skew: bool = False) -> np.ndarray:
    """counts[s, d] = tokens of rank s whose two largest logits include d."""
    first, second = moe_top2_routing(seed, P, tokens, skew)
    counts = np.zeros((P, P), dtype=np.int64)
    for s in range(P):
        counts[s] = np.bincount(first[s], minlength=P) + np.bincount(second[s], minlength=P)
    return counts


def moe_row_maps(first: np.ndarray, second: np.ndarray):
    """Row maps of a token dispatch with packed buffers.

    ``gather[j]``: the global token row (rank * tokens + token) that row j of the
    packed send buffer holds: every rank's rows sorted by destination, ascending
    token order inside a block.  ``scatter[j]``: where row j of the packed receive
    buffer (grouped by source rank) goes in the expert's own order: sorted by
    token index first, source rank second.  Both as int64 arrays of length
    2 * P * tokens."""
    P, tokens = first.shape
    gather = np.empty(2 * P * tokens, dtype=np.int64)
    dest = np.empty(2 * P * tokens, dtype=np.int64)
    for s in range(P):
        d = np.concatenate([first[s], second[s]])
        t = np.concatenate([np.arange(tokens), np.arange(tokens)])
        order = np.lexsort((t, d))                       # by destination, then token
        gather[2 * s * tokens:2 * (s + 1) * tokens] = s * tokens + t[order]
        dest[2 * s * tokens:2 * (s + 1) * tokens] = d[order]
    # receive side: rows of rank d in (source, position) order are the send rows with
    # destination d in ascending send position
    send_pos = np.arange(2 * P * tokens)
    recv_order = np.lexsort((send_pos, dest))            # receive row j holds send row recv_order[j]
    tok = gather[recv_order] % tokens
    src = gather[recv_order] // tokens
    rdest = dest[recv_order]
    expert_order = np.lexsort((src, tok, rdest))         # by receiver, then token, then source
    scatter = np.empty_like(expert_order)
    scatter[expert_order] = np.arange(2 * P * tokens)
    return gather, scatter


def make_c4(seed: int | None = None, P: int = 64, tokens: int = 8192, hidden: int = 4096,
            skew: bool = False) -> Workload:
    seed = bench_seed(4) if seed is None else seed
    c = moe_top2_counts(seed, P, tokens, skew)
    return _finish("c4" + ("_skew" if skew else ""), P, 2 * hidden, seed, c,
                   radices=tuple(r for r in (2, 8, 64) if r <= P))


def make_c5(seed: int | None = None, P: int = 2048, max_bytes: int = 512,
            zero_frac: float = 0.3, hier: tuple | None = (32, 64),
            gaps: bool = False) -> Workload:
    seed = bench_seed(5) if seed is None else seed
    c = uniform_int(seed, S_COUNTS, P * P, 0, max_bytes).numpy()
    z = uniform_unit(seed, S_ZERO, P * P).numpy() < zero_frac
    c = np.where(z, 0, c).reshape(P, P)
    if hier is not None and hier[0] * hier[1] != P:
        hier = None
    return _finish("c5", P, 1, seed, c, gaps=gaps,
                   radices=tuple(r for r in (2, 8, 32, P) if r <= P), hier=hier,
                   hier_radices=tuple(dict.fromkeys(
                       [(hier[0], hier[1])] + [(a, b) for a in (2, 8, 32) for b in (2, 8, 64)
                                               if a <= max(2, hier[0]) and b <= max(2, hier[1])]))
                   if hier else ())


def make_uniform(P: int, count: int, elem_size: int = 1, seed: int = 7) -> Workload:
    """All blocks the same size (the uniform exchange the classic algorithm assumes)."""
    return _finish("uniform", P, elem_size, seed, np.full((P, P), count, dtype=np.int64))


def make_random(P: int, max_count: int, elem_size: int = 1, seed: int = 11,
                zero_frac: float = 0.0, gaps: bool = False) -> Workload:
    c = uniform_int(seed, S_COUNTS, P * P, 0, max_count).numpy()
    if zero_frac > 0:
        c = np.where(uniform_unit(seed, S_ZERO, P * P).numpy() < zero_frac, 0, c)
    return _finish("random", P, elem_size, seed, c.reshape(P, P), gaps=gaps)


def make_silent_ranks(P: int, max_count: int, silent_from: int, silent_to: int, deaf_from: int,
                      deaf_to: int, elem_size: int = 1, seed: int = 13, gaps: bool = False) -> Workload:
    """Random counts in which the ranks [silent_from, silent_to) send nothing and the ranks
    [deaf_from, deaf_to) receive nothing: long runs of empty blocks in every list."""
    c = uniform_int(seed, S_COUNTS, P * P, 0, max_count).numpy().reshape(P, P).copy()
    c[silent_from:silent_to, :] = 0
    c[:, deaf_from:deaf_to] = 0
    return _finish("silent_ranks", P, elem_size, seed, c, gaps=gaps)


# ---- the paper's other count patterns (Sec. VI-A and VI-C), all closed-form or seeded ----

def make_normal(seed: int | None = None, P: int = 4096, mean: float = 1000.0, sd: float = 240.0,
                cap: int = 1024) -> Workload:
    """Block sizes N(mean, sd) in bytes, clipped to [0, cap] (Sec. VI-C: mean 1000,
    standard deviation 240, blocks of at most 1024 bytes, P = 4096)."""
    seed = bench_seed(6) if seed is None else seed
    u1 = uniform_unit(seed, S_COUNTS, P * P).numpy()
    u2 = uniform_unit(seed, S_ZERO, P * P).numpy()
    z = np.sqrt(-2.0 * np.log(1.0 - u1)) * np.cos(2.0 * math.pi * u2)
    c = np.clip(np.rint(mean + sd * z), 0, cap).astype(np.int64).reshape(P, P)
    return _finish("normal", P, 1, seed, c, radices=tuple(r for r in (2, 64, P) if r <= P))


def make_powerlaw(seed: int | None = None, P: int = 4096, exponent: float = 0.95,
                  cap: int = 1024) -> Workload:
    """Block sizes with Pr[c] proportional to (c+1)^-exponent on {0..cap} bytes
    (Sec. VI-C: exponent 0.95; large blocks are rare, many are empty or tiny)."""
    seed = bench_seed(7) if seed is None else seed
    c = zipf_counts(seed, P * P, exponent, cap).reshape(P, P)
    return _finish("powerlaw", P, 1, seed, c, radices=tuple(r for r in (2, 64, P) if r <= P))


def make_fft_n1(P: int = 4096) -> Workload:
    """FFT transpose with N1 = ceil(0.78125 P) * ceil(0.625 P) * 8 (Sec. VI-A): the
    ranks below ceil(0.625 P) each send 8 FP64 values in each of their first
    ceil(0.78125 P) blocks; everything else is empty."""
    workers, filled = math.ceil(0.625 * P), math.ceil(0.78125 * P)
    c = np.zeros((P, P), dtype=np.int64)
    c[:workers, :filled] = 8
    return _finish("fft_n1", P, 8, bench_seed(8), c, radices=tuple(r for r in (2, 64, P) if r <= P))


def make_fft_n2(P: int = 4096) -> Workload:
    """FFT transpose with N2 = ((P-1) * 32 + 8) * P complex values (Sec. VI-A): per
    sender P-1 blocks of 32 complex = 64 FP64 values and a last block of 8 complex
    = 16 FP64 values."""
    c = np.full((P, P), 64, dtype=np.int64)
    c[:, P - 1] = 16
    return _finish("fft_n2", P, 8, bench_seed(9), c, radices=tuple(r for r in (2, 64, P) if r <= P))


FULL = {"c1": make_c1, "c2": make_c2, "c3": make_c3, "c4": make_c4, "c5": make_c5,
        "normal": make_normal, "powerlaw": make_powerlaw, "fft_n1": make_fft_n1,
        "fft_n2": make_fft_n2}
