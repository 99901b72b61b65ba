"""Exact rational arithmetic with explicit IEEE roundings, for brute-force pins.

Nothing here calls the oracle or the CUDA library.  Values are
``fractions.Fraction``; ``round_to`` rounds a rational to the nearest number
representable with ``p`` significant bits and minimum exponent ``emin``
(ties to even), which is what one IEEE operation does to its exact result.
"""
from fractions import Fraction
import struct

F32 = dict(p=24, emin=-126)     # binary32
BF16 = dict(p=8, emin=-126)     # bfloat16: same exponent range, 8 significant bits


def rint_even(q: Fraction) -> int:
    """Nearest integer, ties to even."""
    fl = q.numerator // q.denominator
    rem = q - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        return fl + 1
    return fl


def round_to(q: Fraction, p: int, emin: int) -> Fraction:
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    # exponent e with 2^e <= a < 2^(e+1)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    elif Fraction(2) ** (e + 1) <= a:
        e += 1
    e = max(e, emin)                       # subnormals share the spacing of emin
    ulp = Fraction(2) ** (e - (p - 1))
    return sign * rint_even(a / ulp) * ulp


def f32(q):
    return round_to(Fraction(q), **F32)


def bf16(q):
    return round_to(Fraction(q), **BF16)


def frac_from_bf16_word(h: int) -> Fraction:
    (f,) = struct.unpack("<f", struct.pack("<I", (h & 0xFFFF) << 16))
    return Fraction(f)


def bf16_word(q: Fraction) -> int:
    """Raw bf16 word of a value that is exactly representable in bf16."""
    (u,) = struct.unpack("<I", struct.pack("<f", float(q)))
    assert u & 0xFFFF == 0, "not a bf16 value"
    return u >> 16


def f32_word(q: Fraction) -> int:
    (u,) = struct.unpack("<I", struct.pack("<f", float(q)))
    assert Fraction(struct.unpack("<f", struct.pack("<I", u))[0]) == q, "not an fp32 value"
    return u


# FP8 formats: significand bits, minimum exponent, largest finite value, flush threshold
FP8 = {"e4m3": dict(p=4, emin=-6, fmax=Fraction(448), flush=Fraction(2) ** -117),
       "e5m2": dict(p=3, emin=-14, fmax=Fraction(57344), flush=Fraction(2) ** -110)}


def quantize_block_fp8(v, fmt):
    """v: Fractions that are fp32 values -> (scale, code VALUES as Fractions)."""
    f = FP8[fmt]
    amax = max(abs(t) for t in v)
    if amax < f["flush"]:
        return Fraction(0), [Fraction(0)] * len(v)
    scale = f32(amax / f["fmax"])
    inv = f32(f["fmax"] / amax)
    vals = []
    for t in v:
        r = round_to(f32(t * inv), f["p"], f["emin"])
        vals.append(max(-f["fmax"], min(f["fmax"], r)))
    return scale, vals


def quantize_block(v):
    """v: list of Fractions that are fp32 values -> (scale Fraction, codes list[int])."""
    amax = max(abs(t) for t in v)
    if amax < Fraction(2) ** -118:
        return Fraction(0), [0] * len(v)
    scale = f32(amax / 127)
    inv = f32(Fraction(127) / amax)
    codes = [max(-127, min(127, rint_even(f32(t * inv)))) for t in v]
    return scale, codes


def chain_allreduce(words, block, payload="int8"):
    """words[r][i]: bf16 words, N ranks x count.  Per-shard adder chains.

    Shard k is reduced along ranks k+1, k+2, ..., k (mod N); every link
    quantizes, the next rank dequantizes with one fused multiply-add.
    Returns (out_words[count], events) with events[(k, b, j)] = (scale, codes).
    """
    n_ranks = len(words)
    count = len(words[0])
    shard = count // n_ranks
    out = [0] * count
    events = {}
    for k in range(n_ranks):
        for b in range(shard // block):
            idx = [k * shard + b * block + i for i in range(block)]
            order = [(k + 1 + j) % n_ranks for j in range(n_ranks)]
            v = [frac_from_bf16_word(words[order[0]][i]) for i in idx]
            for j in range(n_ranks):
                scale, codes = quantize_block(v) if payload == "int8" else quantize_block_fp8(v, payload)
                events[(k, b, j)] = (scale, codes)
                if j < n_ranks - 1:
                    nxt = order[j + 1]
                    v = [f32(c * scale + frac_from_bf16_word(words[nxt][i]))
                         for c, i in zip(codes, idx)]
            for c, i in zip(codes, idx):
                out[i] = bf16_word(bf16(f32(c * scale)))
    return out, events


def _quantize(v, payload):
    """(scale, code VALUES as Fractions) for any payload."""
    if payload == "int8":
        scale, codes = quantize_block(v)
        return scale, [Fraction(c) for c in codes]
    return quantize_block_fp8(v, payload)


def tree_allreduce(words, block, semi, quant_rs, quant_ag, payload="int8"):
    """The adder chain of Fig. 4 (semi = False) or the adder tree of Fig. 5 (semi = True) of
    every shard, with or without quantized reduce-scatter hops and all-gather (Section 3.4).

    A hop is `send(v)` followed by `receive(message, addend)`:
      quantized  : message = (scale, codes) of v; result = f32(code * scale + addend), ONE rounding,
                   and the result stays an fp32 value until it is sent again;
      unquantized: message = bf16(v); result = bf16(message + addend).
    Semi loop, shard k, h = N/2 (Section 3.3: on four devices 2 -> 1 -> 0 and 3 -> 0):
      chain A: k+h -> k+h-1 -> ... -> k+1 -> owner k      (h hops, events 0..h-1)
      chain B: k+h+1 -> k+h+2 -> ... -> k-1 -> owner k    (h-1 hops, events h..N-2)
      B is one hop shorter, so its partial reaches the owner first: the owner holds its own shard,
      receives B's message, then A's.
    All-gather: one more quantize/dequantize pair (event N-1), or a plain bf16 rounding.
    Returns (out_words, events) with events[(k, b, j)] = (scale, code values).  Rationals have no
    signed zero: a result that is -0.0 in IEEE arithmetic comes back as the word 0x0000.
    """
    n_ranks = len(words)
    count = len(words[0])
    shard = count // n_ranks
    h = n_ranks // 2
    out = [0] * count
    events = {}
    for k in range(n_ranks):
        for b in range(shard // block):
            idx = [k * shard + b * block + i for i in range(block)]

            def x(rank):
                return [frac_from_bf16_word(words[rank % n_ranks][i]) for i in idx]

            def hop(v, addend, event):
                if quant_rs:
                    scale, vals = _quantize(v, payload)
                    events[(k, b, event)] = (scale, vals)
                    return [f32(c * scale + a) for c, a in zip(vals, addend)]
                return [bf16(bf16(t) + a) for t, a in zip(v, addend)]

            if not semi:
                v = x(k + 1)
                for j in range(1, n_ranks):
                    v = hop(v, x(k + 1 + j), j - 1)
                acc = v
            else:
                acc = x(k)                                  # the owner's own shard
                if h >= 2:                                  # chain B, received first
                    v = x(k + h + 1)
                    for j in range(1, h - 1):
                        v = hop(v, x(k + h + 1 + j), h + j - 1)
                    acc = hop(v, acc, n_ranks - 2)
                v = x(k + h)                                # chain A, received second
                for j in range(1, h):
                    v = hop(v, x(k + h - j), j - 1)
                acc = hop(v, acc, h - 1)
            if quant_ag:
                scale, vals = _quantize(acc, payload)
                events[(k, b, n_ranks - 1)] = (scale, vals)
                res = [bf16(f32(c * scale)) for c in vals]
            else:
                res = [bf16(t) for t in acc]
            for r, i in zip(res, idx):
                out[i] = bf16_word(r)
    return out, events
