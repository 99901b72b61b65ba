// sm_100a kernels for the EQuARX hot path: block-wise int8 quantize, the fused
// dequantize / fp32 add / requantize of a ring hop, and the all-gather
// dequantize (arXiv 2506.17615, Sections 3.1, 3.2, 3.4).
//
// Thread mapping, shared by every kernel: one lane owns 16 contiguous
// elements (one 256-bit bf16 access, one 128-bit int8 access), so a block of
// B elements is B/16 neighbouring lanes of one warp and the per-block max is
// an in-lane max followed by log2(B/16) shuffles.
//
// Kernel families, all bit-identical in their results:
//   rs_step_kernel, ag_dequant_kernel   one launch per ring step over all simulated ranks
//                                       (grid.y = rank or shard, grid.x tiles the shard)
//   pipelined_kernel, flavour_kernel    one persistent launch, every message written as a record
//   chain_fused_kernel, flavour_fused_kernel   one persistent launch, messages kept in registers
//   ring_rank_kernel                    one rank per device: peer mailboxes, per-tile flags
//   bf16_step_kernel, bf16_gather_kernel        the unquantized comparator
//
// Every floating-point step that decides a bit of the result uses an explicit
// round-to-nearest intrinsic, so the compiler cannot contract or reorder it:
//   scale = __fdiv_rn(amax, 127), inv = __fdiv_rn(127, amax)
//   code  = rne(mul.rn(v, inv))       (the add.rn of 1.5*2^23 rounds to the integer grid)
//   hop   = fma.rn((float)code, scale, local)
//   final = cvt.rn.bf16(mul.rn((float)code, scale))
// (mul/add/fma are the packed .f32x2 forms of sm_100: two IEEE results per instruction.)
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace equarx {

constexpr int kThreads = 256;        // threads per CTA of the per-step kernels (64/128/512 measured: not better)
constexpr int kLaneElems = 16;       // elements per lane
constexpr int kMaxRanks = 64;

struct alignas(32) Vec8 {
    uint32_t w[8];
};

// ---------------------------------------------------------------- memory access
// bf16 inputs are read exactly once per step: 256-bit, bypass L1, first to leave L2.
__device__ __forceinline__ Vec8 ld_stream_256(const void* p) {
    Vec8 r;
    asm volatile(
        "ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
        : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]),
          "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
        : "l"(p));
    return r;
}

// bf16 outputs are written once and not read again by this library.
__device__ __forceinline__ void st_stream_256(void* p, const Vec8& r) {
    asm volatile(
        "st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
        ::"l"(p), "r"(r.w[0]), "r"(r.w[1]), "r"(r.w[2]), "r"(r.w[3]),
          "r"(r.w[4]), "r"(r.w[5]), "r"(r.w[6]), "r"(r.w[7])
        : "memory");
}

// Hop messages are written by one step and read by the next: ask L2 to keep them.
// They are read with plain (coherent) loads, never through the read-only path: under
// programmatic dependent launch the reading grid can already be resident while the grid
// before it is still writing those bytes, and the message slots are reused every two steps,
// so the data is not read-only for the lifetime of the reading kernel.  L1 is bypassed.
__device__ __forceinline__ uint64_t policy_keep() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint4 ld_wire_128(const void* p, uint64_t pol) {
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.v4.b32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p), "l"(pol)
                 : "memory");
    return r;
}

__device__ __forceinline__ void st_wire_128(void* p, const uint4& r, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1,%2,%3,%4}, %5;"
                 ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w), "l"(pol)
                 : "memory");
}

__device__ __forceinline__ float ld_scale(const float* p, uint64_t pol) {
    float r;
    asm volatile("ld.global.L1::no_allocate.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(r) : "l"(p), "l"(pol) : "memory");
    return r;
}

__device__ __forceinline__ void st_scale(float* p, float v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
}

// Accessors for data that is written and read inside the SAME launch (the pipelined
// kernels): no read-only (.nc) path.  A record is always stored by the lanes of a warp and,
// after a __syncwarp, loaded by lanes of the same warp, so the loads may use the default
// (L1-allocating) path: the SM's own stores keep its L1 consistent.
__device__ __forceinline__ Vec8 ld_coherent_256(const void* p) {
    Vec8 r;
    asm volatile(
        "ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
        : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]),
          "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
        : "l"(p)
        : "memory");
    return r;
}

__device__ __forceinline__ Vec8 ld_fifo_256(const void* p) {
    Vec8 r;
    asm volatile("ld.global.L1::no_allocate.L2::evict_last.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]),
                   "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                 : "l"(p)
                 : "memory");
    return r;
}

__device__ __forceinline__ void st_fifo_256(void* p, const Vec8& r) {
    asm volatile("st.global.L1::no_allocate.L2::evict_last.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "r"(r.w[0]), "r"(r.w[1]), "r"(r.w[2]), "r"(r.w[3]),
                   "r"(r.w[4]), "r"(r.w[5]), "r"(r.w[6]), "r"(r.w[7])
                 : "memory");
}

__device__ __forceinline__ uint4 ld_coherent_128(const void* p) {
    uint4 r;
    asm volatile("ld.global.ca.v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p)
                 : "memory");
    return r;
}

__device__ __forceinline__ float ld_coherent_f32(const float* p) {
    float r;
    asm volatile("ld.global.ca.f32 %0, [%1];" : "=f"(r) : "l"(p) : "memory");
    return r;
}

__device__ __forceinline__ void st_plain_128(void* p, const uint4& r) {
    asm volatile("st.global.cg.v4.b32 [%0], {%1,%2,%3,%4};"
                 ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w)
                 : "memory");
}

__device__ __forceinline__ void st_plain_f32(float* p, float v) {
    asm volatile("st.global.cg.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

// Programmatic dependent launch: let the next step's CTAs be scheduled while this
// grid drains, and order this grid's dependent reads/writes after the previous grid.
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void pdl_wait_prior_grid() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---------------------------------------------------------------- arithmetic
// sm_100 packed fp32: one instruction, two independent IEEE round-to-nearest results.
// The path is bound by instruction issue as much as by memory, so halving the count of
// the multiplies and adds matters; each half rounds exactly like the scalar intrinsic.
__device__ __forceinline__ void fma2_rn(float& d0, float& d1, float a0, float a1, float b, float c0, float c1) {
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %6};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void mul2_rn(float& d0, float& d1, float a0, float a1, float b) {
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b));
}
__device__ __forceinline__ void add2_rn(float& d0, float& d1, float a0, float a1, float b) {
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1)
        : "f"(a0), "f"(a1), "f"(b));
}

// bf16 -> fp32 is exact: the bf16 word is the upper half of the fp32 word.
__device__ __forceinline__ void widen_bf16x16(const Vec8& x, float (&v)[16]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        v[2 * i] = __uint_as_float(x.w[i] << 16);
        v[2 * i + 1] = __uint_as_float(x.w[i] & 0xFFFF0000u);
    }
}

// int8 -> fp32, exact: byte b (two's complement) xor 0x80 is b+128 in [1, 255]; placed
// in the low mantissa byte of 2^23 it reads 2^23 + b + 128; one exact subtraction
// gives (float)b.  Code 0 gives +0.0f.
__device__ __forceinline__ void codes_to_f32x16(const uint4& c, float (&q)[16]) {
    const uint32_t w[4] = {c.x ^ 0x80808080u, c.y ^ 0x80808080u, c.z ^ 0x80808080u, c.w ^ 0x80808080u};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float u0 = __uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7540));
        const float u1 = __uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7541));
        const float u2 = __uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7542));
        const float u3 = __uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7543));
        add2_rn(q[4 * j + 0], q[4 * j + 1], u0, u1, -8388736.0f);
        add2_rn(q[4 * j + 2], q[4 * j + 3], u2, u3, -8388736.0f);
    }
}

// v[i] = fma((float)code[i], scale, v[i]): the hop's dequantize-and-add, one rounding.
__device__ __forceinline__ void dequant_add_x16(const uint4& c, float scale, float (&v)[16]) {
    float q[16];
    codes_to_f32x16(c, q);
#pragma unroll
    for (int i = 0; i < 8; ++i) fma2_rn(v[2 * i], v[2 * i + 1], q[2 * i], q[2 * i + 1], scale, v[2 * i], v[2 * i + 1]);
}

// bf16x2 words of (float)code[i] * scale, rounded to nearest even: the all-gather dequantize.
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi);
__device__ __forceinline__ Vec8 dequant_to_bf16x16(const uint4& c, float scale) {
    float q[16];
    codes_to_f32x16(c, q);
    Vec8 o;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        mul2_rn(lo, hi, q[2 * i], q[2 * i + 1], scale);
        o.w[i] = pack_bf16x2_rn(lo, hi);
    }
    return o;
}

template <int LPB>
__device__ __forceinline__ float block_max(float m) {
#pragma unroll
    for (int off = LPB / 2; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    return m;
}

// 3-input max (sm_100): halves the instruction count of the in-lane max.
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// Q_p1 + Q_p2 on the 16 values of one lane; the block is LPB neighbouring lanes.
// |v * inv| <= 127 * (1 + 2^-24)^2 < 127.5, so the rounded code never leaves
// [-127, 127] and needs no clamp; adding 1.5 * 2^23 rounds to nearest-even on the
// integer grid and leaves the two's-complement code in the low byte.
// Each lane performs ONE of the block's two IEEE divisions (even lanes amax/127, odd
// lanes 127/amax; the operands are selected, the instruction stream is the same) and
// the pair of lanes exchanges the quotients with two shuffles.
template <int LPB>
__device__ __forceinline__ void block_scale_and_inverse(const float (&v)[16], float& scale, float& inv) {
    float m = max3(fabsf(v[0]), fabsf(v[1]), fabsf(v[2]));
    float m1 = max3(fabsf(v[3]), fabsf(v[4]), fabsf(v[5]));
    float m2 = max3(fabsf(v[6]), fabsf(v[7]), fabsf(v[8]));
    float m3 = max3(fabsf(v[9]), fabsf(v[10]), fabsf(v[11]));
    m = max3(m, fabsf(v[12]), fabsf(v[13]));
    m1 = max3(m1, fabsf(v[14]), fabsf(v[15]));
    m = max3(m, m1, fmaxf(m2, m3));
    m = block_max<LPB>(m);
    const bool odd = threadIdx.x & 1u;
    // a flushed block (amax below 2^-118, zero included) divides 1.0 instead: its quotient is
    // discarded, and the division never leaves its fast path on zeros and subnormals
    const bool live = m >= 0x1p-118f;
    const float ms = live ? m : 1.0f;
    const float quot = __fdiv_rn(odd ? 127.0f : ms, odd ? ms : 127.0f);
    const float keep = live ? quot : 0.0f;                // flush rule: scale = inv = 0
    scale = __shfl_sync(0xFFFFFFFFu, keep, (threadIdx.x & 30u));
    inv = __shfl_sync(0xFFFFFFFFu, keep, (threadIdx.x & 30u) | 1u);
}

template <int LPB>
__device__ __forceinline__ void quantize_lane(const float (&v)[16], uint4& codes, float& scale, float neg_zero) {
    float inv;
    block_scale_and_inverse<LPB>(v, scale, inv);
    uint32_t b[16];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        // The product must be rounded to fp32 BEFORE the add of 1.5 * 2^23 (two roundings, as in
        // rintf(v * inv)).  ptxas contracts a packed mul.rn.f32x2 (or a packed fma with a literal
        // zero addend) feeding a packed add.rn.f32x2 into one fused multiply-add (seen on ties:
        // 63.5 -> 63 instead of 64).  So the product is formed by a packed fma whose addend is
        // -0.0 passed in as a kernel argument: it leaves every product unchanged, the compiler
        // cannot fold it away, and an fma cannot be merged with the following add.
        float t0, t1, r0, r1;
        fma2_rn(t0, t1, v[2 * i], v[2 * i + 1], inv, neg_zero, neg_zero);
        add2_rn(r0, r1, t0, t1, 12582912.0f);
        b[2 * i] = __float_as_uint(r0);
        b[2 * i + 1] = __float_as_uint(r1);
    }
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t lo = __byte_perm(b[4 * j + 0], b[4 * j + 1], 0x0040);
        const uint32_t hi = __byte_perm(b[4 * j + 2], b[4 * j + 3], 0x0040);
        o[j] = __byte_perm(lo, hi, 0x5410);
    }
    codes = make_uint4(o[0], o[1], o[2], o[3]);
}

// The same quantization with every code kept as the fp32 value of the int8 code (an integer in
// [-127, 127]) instead of a packed byte: r = fl(fl(v * inv) + 1.5 * 2^23) holds the code in its
// low mantissa bits, and r - 1.5 * 2^23 is exact and equals (float)code, +0.0 for code 0.  Used
// where the message is consumed by the lane that produced it and never leaves the registers.
template <int LPB>
__device__ __forceinline__ void quantize_lane_values(const float (&v)[16], float (&q)[16], float& scale, float neg_zero) {
    float inv;
    block_scale_and_inverse<LPB>(v, scale, inv);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float t0, t1, r0, r1;
        fma2_rn(t0, t1, v[2 * i], v[2 * i + 1], inv, neg_zero, neg_zero);      // see quantize_lane
        add2_rn(r0, r1, t0, t1, 12582912.0f);
        add2_rn(q[2 * i], q[2 * i + 1], r0, r1, -12582912.0f);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// ---------------------------------------------------------------- FP8 payloads
// The same block-wise rule with the format's largest finite value in place of 127
// (E4M3: 448, E5M2: 57344); codes are produced by the hardware conversion
// cvt.rn.satfinite.{e4m3x2,e5m2x2}.f32 and widened again through f16, which holds every
// FP8 value exactly.  PAYLOAD: 1 int8, 2 E4M3, 3 E5M2.
template <int PAYLOAD> struct Fp8Format;
template <> struct Fp8Format<2> { static constexpr float kMax = 448.0f, kFlush = 0x1p-117f; };
template <> struct Fp8Format<3> { static constexpr float kMax = 57344.0f, kFlush = 0x1p-110f; };

template <int PAYLOAD>
__device__ __forceinline__ uint32_t f32x2_to_fp8x2(float lo, float hi) {
    uint16_t d;
    if (PAYLOAD == 2) asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    else asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

template <int PAYLOAD>
__device__ __forceinline__ void fp8x4_to_f32(uint32_t w, float& f0, float& f1, float& f2, float& f3) {
    uint32_t h01, h23;
    if (PAYLOAD == 2) {
        asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(w));
    } else {
        asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e5m2x2 %0, a;\n\tcvt.rn.f16x2.e5m2x2 %1, b;\n\t}"
            : "=r"(h01), "=r"(h23) : "r"(w));
    }
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}"
        : "=f"(f0), "=f"(f1) : "r"(h01));
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}"
        : "=f"(f2), "=f"(f3) : "r"(h23));
}

// payload bytes -> fp32, exact
template <int PAYLOAD>
__device__ __forceinline__ void decode_x16(const uint4& c, float (&q)[16]) {
    if (PAYLOAD == 1) {
        codes_to_f32x16(c, q);
    } else {
        fp8x4_to_f32<PAYLOAD>(c.x, q[0], q[1], q[2], q[3]);
        fp8x4_to_f32<PAYLOAD>(c.y, q[4], q[5], q[6], q[7]);
        fp8x4_to_f32<PAYLOAD>(c.z, q[8], q[9], q[10], q[11]);
        fp8x4_to_f32<PAYLOAD>(c.w, q[12], q[13], q[14], q[15]);
    }
}

// the block quantizer for any payload (PAYLOAD 1 is quantize_lane)
template <int LPB, int PAYLOAD>
__device__ __forceinline__ void quantize_lane_payload(const float (&v)[16], uint4& codes, float& scale, float neg_zero) {
    if (PAYLOAD == 1) {
        quantize_lane<LPB>(v, codes, scale, neg_zero);
        return;
    }
    constexpr int F = PAYLOAD == 1 ? 2 : PAYLOAD;
    float m = max3(fabsf(v[0]), fabsf(v[1]), fabsf(v[2]));
    float m1 = max3(fabsf(v[3]), fabsf(v[4]), fabsf(v[5]));
    float m2 = max3(fabsf(v[6]), fabsf(v[7]), fabsf(v[8]));
    float m3 = max3(fabsf(v[9]), fabsf(v[10]), fabsf(v[11]));
    m = max3(m, fabsf(v[12]), fabsf(v[13]));
    m1 = max3(m1, fabsf(v[14]), fabsf(v[15]));
    m = max3(m, m1, fmaxf(m2, m3));
    m = block_max<LPB>(m);
    const bool odd = threadIdx.x & 1u;
    const bool live = m >= Fp8Format<F>::kFlush;
    const float ms = live ? m : 1.0f;
    const float quot = __fdiv_rn(odd ? Fp8Format<F>::kMax : ms, odd ? ms : Fp8Format<F>::kMax);
    const float keep = live ? quot : 0.0f;
    scale = __shfl_sync(0xFFFFFFFFu, keep, (threadIdx.x & 30u));
    const float inv = __shfl_sync(0xFFFFFFFFu, keep, (threadIdx.x & 30u) | 1u);
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float t0, t1, t2, t3;
        mul2_rn(t0, t1, v[4 * j + 0], v[4 * j + 1], inv);
        mul2_rn(t2, t3, v[4 * j + 2], v[4 * j + 3], inv);
        o[j] = f32x2_to_fp8x2<F>(t0, t1) | (f32x2_to_fp8x2<F>(t2, t3) << 16);
    }
    codes = make_uint4(o[0], o[1], o[2], o[3]);
}

template <int PAYLOAD>
__device__ __forceinline__ void dequant_add_payload(const uint4& c, float scale, float (&v)[16]) {
    float q[16];
    decode_x16<PAYLOAD>(c, q);
#pragma unroll
    for (int i = 0; i < 8; ++i) fma2_rn(v[2 * i], v[2 * i + 1], q[2 * i], q[2 * i + 1], scale, v[2 * i], v[2 * i + 1]);
}

template <int PAYLOAD>
__device__ __forceinline__ Vec8 dequant_to_bf16_payload(const uint4& c, float scale) {
    float q[16];
    decode_x16<PAYLOAD>(c, q);
    Vec8 o;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float lo, hi;
        mul2_rn(lo, hi, q[2 * i], q[2 * i + 1], scale);
        o.w[i] = pack_bf16x2_rn(lo, hi);
    }
    return o;
}

// ---------------------------------------------------------------- message layouts
// SPLIT   (the per-step entry points): codes[count] and scales[count/B] are separate arrays.
// RECORDS (the simulations): a message is a sequence of 544-byte records, one per tile of
//         512 elements: 8 floats of metadata first (the tile's 512/B scales, zero padded to
//         one 32-byte sector), then the 512 codes (Section 3.1 sends metadata ahead of
//         the microshards it describes).  Every sector of a record is written whole, so a
//         message that is read back while it is still in L2 never needs a fill from DRAM.
constexpr int kTileElems = 512;
constexpr int kRecordHeader = 32;
constexpr int kRecordBytes = kRecordHeader + kTileElems;

template <int LPB>
__device__ __forceinline__ void st_record(char* rec, uint32_t lane, bool lane_active, bool tile_active,
                                          const uint4& codes, float scale, uint64_t pol) {
    // lanes 0..7 write the header sector: lane i holds the scale of block i of the tile
    float hdr = __shfl_sync(0xFFFFFFFFu, scale, (lane * LPB) & 31u);
    if (lane >= 32u / LPB) hdr = 0.0f;
    if (tile_active && lane < 8) st_scale(reinterpret_cast<float*>(rec) + lane, hdr, pol);
    if (lane_active) st_wire_128(rec + kRecordHeader + lane * 16, codes, pol);
}

// ---------------------------------------------------------------- kernel arguments
// One launch covers every simulated rank.  Messages live in "slots".
struct StepArgs {
    const void* x[kMaxRanks];        // rank r's bf16 shard for this step
    uint32_t in_slot[kMaxRanks];     // message received by rank r (unused at step 0)
    uint32_t out_slot[kMaxRanks];    // message produced by rank r
    const int8_t* codes_in;          // SPLIT: codes region; RECORDS: record region
    const float* scales_in;          // SPLIT only
    int8_t* codes_out;
    float* scales_out;
    uint64_t shard;                  // elements per message
    uint64_t bps;                    // SPLIT: blocks per message; RECORDS: bytes per slot
    float neg_zero;                  // -0.0f, opaque to the compiler (see quantize_lane)
};

struct GatherArgs {
    void* out[kMaxRanks];            // output tensor of rank r (whole tensor)
    uint32_t slot[kMaxRanks];        // final message of shard k
    const int8_t* codes;
    const float* scales;
    uint64_t shard;
    uint64_t bps;                    // as in StepArgs
    uint32_t nranks;
};

struct PipeArgs {
    const void* in[kMaxRanks];       // input tensor of rank r (whole tensor)
    void* out[kMaxRanks];            // output tensor of rank r
    char* records;                   // the trace: record region [shard k][event j][tile] (unused by the chain-fused form)
    uint64_t shard;
    uint64_t tiles_per_shard;        // 512-element tiles per shard (the last one may be ragged)
    uint32_t nranks;
    uint32_t unordered;              // chain-fused form only: do not wait for the stream's earlier work before starting
    float neg_zero;                  // -0.0f, opaque to the compiler (see quantize_lane)
};

struct Bf16StepArgs {
    const void* recv[kMaxRanks];     // bf16 shard received by rank r
    const void* local[kMaxRanks];    // rank r's own counterpart
    void* send[kMaxRanks];           // bf16 shard rank r forwards
    uint64_t shard;
};

struct Bf16GatherArgs {
    const void* src[kMaxRanks];      // reduced shard k
    void* out[kMaxRanks];
    uint64_t shard;
    uint32_t nranks;
};

// ---------------------------------------------------------------- kernels
// Ring step: FIRST = step 0 (quantize only), else dequantize-add-requantize.
// Every launch may be a programmatic dependent of the kernel before it in the stream.  Step 0
// reads tensors that the work before it may still be writing (an in-place all-gather, the
// caller's producer), so it waits for that work before its first load; the later steps load
// their bf16 shard, which nothing in this call writes before the all-gather, ahead of the wait.
// 8 CTAs of 256 threads per SM (32 registers, full occupancy): 2-3 % faster than the 34 registers and
// 7 CTAs the compiler picks on its own (B200, 16 MB and 88 MB per rank).
template <int LPB, bool FIRST, bool RECORDS>
__global__ void __launch_bounds__(kThreads, 2048 / kThreads) rs_step_kernel(const __grid_constant__ StepArgs a) {
    const uint32_t r = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;   // 16-element group
    const uint64_t groups = a.shard >> 4;
    const bool active = g < groups;
    const uint64_t pol = policy_keep();

    if (FIRST) pdl_wait_prior_grid();
    Vec8 xw = {};
    if (active) xw = ld_stream_256(static_cast<const char*>(a.x[r]) + g * 32);
    pdl_launch_dependents();

    float v[16];
    widen_bf16x16(xw, v);
    if (!FIRST) {
        pdl_wait_prior_grid();       // the received message comes from the previous launch
        uint4 c = make_uint4(0, 0, 0, 0);
        float s = 0.0f;
        if (active) {
            const uint64_t slot = a.in_slot[r];
            if (RECORDS) {
                const char* rec = reinterpret_cast<const char*>(a.codes_in) + slot * a.bps + (g >> 5) * kRecordBytes;
                c = ld_wire_128(rec + kRecordHeader + lane * 16, pol);
                s = ld_scale(reinterpret_cast<const float*>(rec) + lane / LPB, pol);
            } else {
                c = ld_wire_128(a.codes_in + slot * a.shard + g * 16, pol);
                s = ld_scale(a.scales_in + slot * a.bps + g / LPB, pol);
            }
        }
        dequant_add_x16(c, s, v);
    }

    uint4 codes;
    float scale;
    quantize_lane<LPB>(v, codes, scale, a.neg_zero);
    const uint64_t slot = a.out_slot[r];
    if (RECORDS) {
        char* rec = reinterpret_cast<char*>(a.codes_out) + slot * a.bps + (g >> 5) * kRecordBytes;
        st_record<LPB>(rec, lane, active, (g - lane) < groups, codes, scale, pol);
    } else if (active) {
        st_wire_128(a.codes_out + slot * a.shard + g * 16, codes, pol);
        if ((threadIdx.x & (LPB - 1)) == 0) st_scale(a.scales_out + slot * a.bps + g / LPB, scale, pol);
    }
}

// All-gather receive side: one read of shard k's final message, nranks bf16 writes.
template <int LPB, bool RECORDS>
__global__ void __launch_bounds__(kThreads) ag_dequant_kernel(const __grid_constant__ GatherArgs a) {
    const uint32_t k = blockIdx.y;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool active = g < (a.shard >> 4);
    const uint64_t pol = policy_keep();
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    if (!active) return;
    const uint64_t slot = a.slot[k];
    uint4 c;
    float s;
    if (RECORDS) {
        const char* rec = reinterpret_cast<const char*>(a.codes) + slot * a.bps + (g >> 5) * kRecordBytes;
        c = ld_wire_128(rec + kRecordHeader + lane * 16, pol);
        s = ld_scale(reinterpret_cast<const float*>(rec) + lane / LPB, pol);
    } else {
        c = ld_wire_128(a.codes + slot * a.shard + g * 16, pol);
        s = ld_scale(a.scales + slot * a.bps + g / LPB, pol);
    }
    const Vec8 o = dequant_to_bf16x16(c, s);
    const uint64_t byte_off = (k * a.shard + g * 16) * 2;
    for (uint32_t r = 0; r < a.nranks; ++r) st_stream_256(static_cast<char*>(a.out[r]) + byte_off, o);
}

// Deep-pipelined form of the whole schedule with every message kept (Section 3.1 pipelines the
// microshards of a shard through the ring independently; here a microshard is one tile of 512
// elements).  One warp carries its tile through all N ring steps and the all-gather without
// waiting for any other tile.  Every hop message goes through memory as a record of the trace:
// the lane that acts for the sending rank stores its codes (and lanes 0..7 the metadata sector),
// the warp synchronises, and the NEIGHBOURING lane (lane ^ 1), acting for the receiving rank,
// loads them back and continues with that 16-element group.  The bf16 shard of the next step is
// prefetched while a step computes.
constexpr int kPipeThreads = 64;
#ifndef EQX_PIPE_MINBLOCKS
#define EQX_PIPE_MINBLOCKS 18
#endif

template <int LPB>
__global__ void __launch_bounds__(kPipeThreads, EQX_PIPE_MINBLOCKS) pipelined_kernel(const __grid_constant__ PipeArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps = (uint64_t)gridDim.x * (kPipeThreads / 32);
    const uint64_t warp = (uint64_t)blockIdx.x * (kPipeThreads / 32) + (threadIdx.x >> 5);
    const uint32_t N = a.nranks;
    const uint64_t groups = a.shard >> 4;
    const uint64_t tiles = a.tiles_per_shard * N;
    const uint64_t trace_stride = a.tiles_per_shard * kRecordBytes;      // one event further in the trace
    // byte offsets inside a record: even steps send from position `lane` and receive (as the
    // neighbouring lane, acting for the receiving rank) at position lane ^ 1; odd steps the reverse
    const uint32_t code_own = kRecordHeader + lane * 16, code_nbr = kRecordHeader + (lane ^ 1u) * 16;
    const uint32_t scale_own = (lane / LPB) * 4, scale_nbr = ((lane ^ 1u) / LPB) * 4;
    const uint32_t hdr_src_even = (lane * LPB) & 31u, hdr_src_odd = hdr_src_even ^ 1u;

    // Launched as a programmatic dependent: the grid may be scheduled while the previous kernel of
    // the stream drains, but touches no memory before that kernel has completed and flushed.
    pdl_launch_dependents();
    pdl_wait_prior_grid();

    // byte offset of this lane's own group of a tile in every rank's tensor (the neighbouring group
    // is 32 bytes to the other side); ~0 if the lane is past the end of a ragged last tile
    auto own_offset = [&](uint64_t tile_, uint32_t& k_) -> uint64_t {
        k_ = (uint32_t)(tile_ / a.tiles_per_shard);
        const uint64_t t_ = tile_ - (uint64_t)k_ * a.tiles_per_shard;
        if (t_ * 32 + lane >= groups) return ~uint64_t(0);
        return ((uint64_t)k_ * a.shard + (t_ * 32 + lane) * 16) * 2;
    };
    // the first shard of a tile is fetched while the previous tile finishes (the last step needs
    // no prefetch of its own, so the same registers are free)
    uint32_t k_next = 0;
    uint64_t off_next = warp < tiles ? own_offset(warp, k_next) : ~uint64_t(0);
    Vec8 xw = {};
    if (off_next != ~uint64_t(0))
        xw = ld_coherent_256(static_cast<const char*>(a.in[k_next + 1 == N ? 0 : k_next + 1]) + off_next);

    for (uint64_t tile = warp; tile < tiles; tile += warps) {
        const uint32_t k = k_next;
        const uint64_t off_own = off_next;
        const bool active = off_own != ~uint64_t(0);   // lane pairs are in or out together (groups % 4 == 0)
        const uint64_t off_nbr = off_own ^ 32;         // the neighbouring lane's group
        char* trace = a.records + ((uint64_t)k * N * a.tiles_per_shard + (tile - (uint64_t)k * a.tiles_per_shard)) * kRecordBytes;
        uint32_t rho = k + 1 == N ? 0 : k + 1;         // rank of step 0
        float v[16];
        widen_bf16x16(xw, v);

        // next shard (or, at the last step, the first shard of this warp's next tile)
        auto prefetch = [&](uint32_t j, uint64_t off) {
            rho = rho + 1 == N ? 0 : rho + 1;
            if (j + 1 < N) {
                if (active) xw = ld_coherent_256(static_cast<const char*>(a.in[rho]) + off);
            } else {
                xw = Vec8{};
                off_next = tile + warps < tiles ? own_offset(tile + warps, k_next) : ~uint64_t(0);
                if (off_next != ~uint64_t(0))
                    xw = ld_coherent_256(static_cast<const char*>(a.in[k_next + 1 == N ? 0 : k_next + 1]) + off_next);
            }
        };
        // one ring step: quantize v, send the record, receive it as the neighbouring lane
        auto exchange = [&](char* rec, uint32_t hdr_src, uint32_t code_send, uint32_t code_recv, uint32_t scale_recv,
                            uint4& c, float& s) {
            uint4 codes;
            float scale;
            quantize_lane<LPB>(v, codes, scale, a.neg_zero);
            float hdr = __shfl_sync(0xFFFFFFFFu, scale, hdr_src);       // lanes 0..7 write the metadata sector
            if (lane >= 32u / LPB) hdr = 0.0f;
            if (lane < 8) st_plain_f32(reinterpret_cast<float*>(rec) + lane, hdr);
            if (active) st_plain_128(rec + code_send, codes);
            __syncwarp();                              // the message is now visible to the neighbouring lane
            c = make_uint4(0, 0, 0, 0);
            s = 0.0f;
            if (active) {
                c = ld_coherent_128(rec + code_recv);
                s = ld_coherent_f32(reinterpret_cast<const float*>(rec + scale_recv));
            }
        };
        auto gather = [&](const uint4& c, float s, uint64_t off) {      // all-gather: one store per rank
            const Vec8 o = dequant_to_bf16x16(c, s);
            if (active)
                for (uint32_t r = 0; r < N; ++r) st_stream_256(static_cast<char*>(a.out[r]) + off, o);
        };

        for (uint32_t j = 0;; j += 2) {
            uint4 c;
            float s;
            // even step: send from the own position, receive at the neighbour's
            prefetch(j, off_nbr);
            exchange(trace, hdr_src_even, code_own, code_nbr, scale_nbr, c, s);
            if (j + 1 == N) {
                gather(c, s, off_nbr);
                break;
            }
            widen_bf16x16(xw, v);
            dequant_add_x16(c, s, v);
            trace += trace_stride;
            // odd step: send from the neighbour's position, receive at the own
            prefetch(j + 1, off_own);
            exchange(trace, hdr_src_odd, code_nbr, code_own, scale_own, c, s);
            if (j + 2 == N) {
                gather(c, s, off_own);
                break;
            }
            widen_bf16x16(xw, v);
            dequant_add_x16(c, s, v);
            trace += trace_stride;
        }
    }
}

// Chain-fused form of the same schedule, used when no trace is kept.  A tile's adder chain
// (Section 3.3, Fig. 4) depends on no other tile, so the lane that quantized a 16-element group
// for the sending rank can go on, as the receiving rank, with the fused multiply-add on that
// rank's counterpart: the hop message of a group (its codes, as the fp32 values of the int8
// codes, and the block's scale) stays in that lane's registers and is never stored.  Codes,
// scales and outputs are bit for bit those of pipelined_kernel<LPB>, which writes every
// message as a record and is the witness of that; what this kernel moves through HBM is the
// bf16 inputs once and the bf16 outputs once (4 bytes per element of every rank).
// The bf16 shard of the next rank of the chain is in flight while a step computes; DEPTH is the
// number of such loads in flight per lane.
// MINB = resident CTAs per SM the register allocation aims for.  Measured on B200: 18 (56 registers,
// 36 warps per SM) is faster while the whole AllReduce moves little (below about 200 MB of input: the
// launch is short and more warps fill the memory pipeline sooner), 16 (64 registers, 32 warps) is 2-5 %
// faster above that.  The host picks per launch.
constexpr int kFusedDepth = 1;

// QUANT = false is the unquantized comparator in the same form: the message is the partial sum
// rounded to bf16 and the receiving rank's add is rounded to bf16 again (the BF16 baseline's hop).
template <int LPB, int DEPTH, bool QUANT, int MINB>
__global__ void __launch_bounds__(kPipeThreads, MINB) chain_fused_kernel(const __grid_constant__ PipeArgs a) {
    static_assert(DEPTH == 1 || DEPTH == 2, "one or two shards in flight");
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps = (uint64_t)gridDim.x * (kPipeThreads / 32);
    const uint64_t warp = (uint64_t)blockIdx.x * (kPipeThreads / 32) + (threadIdx.x >> 5);
    const uint32_t N = a.nranks;
    const uint64_t groups = a.shard >> 4;
    const uint64_t tiles = a.tiles_per_shard * N;

    // Ordered (the default): nothing is read before the previous kernel of the stream has completed.
    // Unordered: the caller vouches that no unfinished earlier work of the stream writes the inputs or
    // touches the outputs, so the grid starts while that work is still finishing (this removes the
    // idle gap between back-to-back independent AllReduces) and waits for it only before it exits, so
    // that whatever follows in the stream still sees all earlier work complete.
    pdl_launch_dependents();
    if (!a.unordered) pdl_wait_prior_grid();

    // byte offset of this lane's group of a tile in every rank's tensor; ~0 past the end of a ragged last tile
    auto offset_of = [&](uint64_t tile_, uint32_t& k_) -> uint64_t {
        k_ = (uint32_t)(tile_ / a.tiles_per_shard);
        const uint64_t t_ = tile_ - (uint64_t)k_ * a.tiles_per_shard;
        if (t_ * 32 + lane >= groups) return ~uint64_t(0);
        return ((uint64_t)k_ * a.shard + (t_ * 32 + lane) * 16) * 2;
    };
    auto load = [&](uint32_t rank, uint64_t off) {
        Vec8 x = {};
        if (off != ~uint64_t(0)) x = ld_coherent_256(static_cast<const char*>(a.in[rank]) + off);   // in place is allowed: no read-only path
        return x;
    };
    auto next_rank = [&](uint32_t r) { return r + 1 == N ? 0u : r + 1; };

    // The loads of a tile run over the chain's ranks k+1, k+2, ..., k; when they are used up, the
    // stream of loads continues with the warp's next tile, so DEPTH loads are always in flight.
    uint64_t tile_ld = warp;                    // tile, rank and offset of the next load to issue
    uint32_t k_ld = 0, left_ld = N;             // left_ld: loads of tile_ld still to issue
    uint64_t off_ld = tile_ld < tiles ? offset_of(tile_ld, k_ld) : ~uint64_t(0);
    uint32_t rank_ld = next_rank(k_ld);
    auto issue = [&]() {
        const Vec8 x = load(rank_ld, tile_ld < tiles ? off_ld : ~uint64_t(0));
        rank_ld = next_rank(rank_ld);
        if (--left_ld == 0) {
            tile_ld += warps;
            left_ld = N;
            off_ld = tile_ld < tiles ? offset_of(tile_ld, k_ld) : ~uint64_t(0);
            rank_ld = next_rank(k_ld);
        }
        return x;
    };

    Vec8 x0 = issue(), x1 = {};
    if (DEPTH == 2) x1 = issue();

    for (uint64_t tile = warp; tile < tiles; tile += warps) {
        uint32_t k;
        const uint64_t off = offset_of(tile, k);
        float v[16];                            // the partial sum, then (in place) the code values of its message
        widen_bf16x16(x0, v);                   // rank k+1's shard opens the chain
        if (DEPTH == 2) { x0 = x1; x1 = issue(); } else { x0 = issue(); }
        float scale = 0.0f;
        for (uint32_t j = 1;; ++j) {
            if (QUANT) quantize_lane_values<LPB>(v, v, scale, a.neg_zero);      // the message of step j-1
            if (j == N) break;
            if (QUANT) {
                // the receiving rank: v = fma(code, scale, its counterpart), straight from the bf16 words
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    fma2_rn(v[2 * i], v[2 * i + 1], v[2 * i], v[2 * i + 1], scale,
                            __uint_as_float(x0.w[i] << 16), __uint_as_float(x0.w[i] & 0xFFFF0000u));
            } else {
                // v holds bf16 values (a raw shard, or a rounded sum): the message is v itself
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const uint32_t sum = pack_bf16x2_rn(__fadd_rn(v[2 * i], __uint_as_float(x0.w[i] << 16)),
                                                        __fadd_rn(v[2 * i + 1], __uint_as_float(x0.w[i] & 0xFFFF0000u)));
                    v[2 * i] = __uint_as_float(sum << 16);
                    v[2 * i + 1] = __uint_as_float(sum & 0xFFFF0000u);
                }
            }
            if (DEPTH == 2) { x0 = x1; x1 = issue(); } else { x0 = issue(); }
        }
        // all-gather: the last message, dequantized (or forwarded as it is), goes to every rank
        Vec8 o;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float lo = v[2 * i], hi = v[2 * i + 1];
            if (QUANT) mul2_rn(lo, hi, v[2 * i], v[2 * i + 1], scale);
            o.w[i] = pack_bf16x2_rn(lo, hi);
        }
        if (off != ~uint64_t(0))
            for (uint32_t r = 0; r < N; ++r) st_stream_256(static_cast<char*>(a.out[r]) + off, o);
    }
    if (a.unordered) pdl_wait_prior_grid();
}

// ---------------------------------------------------------------- the other flavours
// Semi-loop ring (Section 3.3, Fig. 5) and stage selection (Section 3.4: quantize the
// reduce-scatter, the all-gather, or both), in the same deep-pipelined form: one warp
// carries a 512-element tile along its adder chain(s); every message goes through the
// warp's two-entry staging FIFO and is read back by the neighbouring lane.  A message
// is a 544-byte quantized record or, for an unquantized stage, 1024 bytes of bf16.
// flavour_kernel is the form used when a trace is kept (every quantized message is also
// written to the trace); flavour_fused_kernel further down keeps the messages in registers.
constexpr int kFifoEntryBytes = 1024;

struct FlavourArgs {
    const void* in[kMaxRanks];
    void* out[kMaxRanks];
    char* fifo;                      // per-warp staging FIFOs (2 entries of kFifoEntryBytes)
    char* trace;                     // record region [shard k][event j][tile], or nullptr
    uint64_t shard;
    uint64_t tiles_per_shard;
    uint32_t nranks;
    float neg_zero;
};

// One hop of a chain, in two halves.  chain_send: the message of v (a quantized record, or bf16
// for an unquantized stage) goes to the FIFO entry (and to the trace), the warp synchronises and
// the lane moves to the neighbouring position (`sub` flips).  chain_receive: the lane, now acting
// for the receiving rank, loads the message and folds it into v_io, which holds the addend: with a
// quantized payload one fused multiply-add in fp32, else an fp32 add rounded to bf16 (the BF16
// baseline's hop).
template <int LPB, int PAYLOAD>
__device__ __forceinline__ void chain_send(const float (&v)[16], char* entry, char* trace_rec, uint32_t lane,
                                           uint32_t& sub, bool active, float neg_zero) {
    if (PAYLOAD != 0) {
        uint4 codes;
        float scale;
        quantize_lane_payload<LPB, PAYLOAD == 0 ? 1 : PAYLOAD>(v, codes, scale, neg_zero);
        const uint32_t d = (sub ^ lane) & 1u;                  // position p is held by lane p ^ d
        float hdr = __shfl_sync(0xFFFFFFFFu, scale, ((lane * LPB) & 31u) ^ d);
        if (lane >= 32u / LPB) hdr = 0.0f;
        if (lane < 8) st_plain_f32(reinterpret_cast<float*>(entry) + lane, hdr);
        if (active) st_plain_128(entry + kRecordHeader + sub * 16, codes);
        if (trace_rec) {                                       // keep the message as well
            if (lane < 8) st_plain_f32(reinterpret_cast<float*>(trace_rec) + lane, hdr);
            if (active) st_plain_128(trace_rec + kRecordHeader + sub * 16, codes);
        }
    } else {
        Vec8 m;
#pragma unroll
        for (int i = 0; i < 8; ++i) m.w[i] = pack_bf16x2_rn(v[2 * i], v[2 * i + 1]);
        if (active) st_fifo_256(entry + sub * 32, m);
    }
    __syncwarp();
    sub ^= 1u;
}

template <int LPB, int PAYLOAD>
__device__ __forceinline__ void chain_receive(float (&v_io)[16], const char* entry, uint32_t sub, bool active) {
    if (PAYLOAD != 0) {
        uint4 c = make_uint4(0, 0, 0, 0);
        float s = 0.0f;
        if (active) {
            c = ld_coherent_128(entry + kRecordHeader + sub * 16);
            s = ld_coherent_f32(reinterpret_cast<const float*>(entry) + sub / LPB);
        }
        dequant_add_payload<PAYLOAD == 0 ? 1 : PAYLOAD>(c, s, v_io);
    } else {
        Vec8 r = {};
        if (active) r = ld_fifo_256(entry + sub * 32);
        float y[16];
        widen_bf16x16(r, y);
        Vec8 o;
#pragma unroll
        for (int i = 0; i < 8; ++i)
            o.w[i] = pack_bf16x2_rn(__fadd_rn(y[2 * i], v_io[2 * i]), __fadd_rn(y[2 * i + 1], v_io[2 * i + 1]));
        widen_bf16x16(o, v_io);
    }
}

template <int LPB, bool SEMI, bool QRS, bool QAG, int PAYLOAD>
__global__ void __launch_bounds__(kPipeThreads) flavour_kernel(const __grid_constant__ FlavourArgs a) {
    constexpr int RS = QRS ? PAYLOAD : 0;          // payload of the reduce-scatter hops (0: bf16 messages)
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps = (uint64_t)gridDim.x * (kPipeThreads / 32);
    const uint64_t warp = (uint64_t)blockIdx.x * (kPipeThreads / 32) + (threadIdx.x >> 5);
    const uint32_t N = a.nranks;
    const uint32_t h = N / 2;
    const uint64_t groups = a.shard >> 4;
    const uint64_t tiles = a.tiles_per_shard * N;
    char* const fifo = a.fifo + warp * (2 * kFifoEntryBytes);

    for (uint64_t tile = warp; tile < tiles; tile += warps) {
        const uint32_t k = (uint32_t)(tile / a.tiles_per_shard);
        const uint64_t t = tile - (uint64_t)k * a.tiles_per_shard;
        const bool active = t * 32 + lane < groups;
        const uint64_t tile_off = (uint64_t)k * a.shard + t * kTileElems;        // first element of the tile
        char* const trace0 = a.trace ? a.trace + ((uint64_t)k * N * a.tiles_per_shard + t) * kRecordBytes : nullptr;
        uint32_t hops = 0;                                                       // FIFO entry = hops & 1

        auto fetch = [&](uint32_t rank, uint32_t pos) {                          // a rank's bf16 group at a position
            Vec8 x = {};
            if (active) x = ld_coherent_256(static_cast<const char*>(a.in[rank % N]) + (tile_off + pos * 16) * 2);
            return x;
        };
        auto trace_of = [&](uint32_t event) -> char* {
            return trace0 ? trace0 + (uint64_t)event * a.tiles_per_shard * kRecordBytes : nullptr;
        };
        // one hop: v is sent; the receiver's addend is either the prefetched shard xw (then the result
        // replaces v) or the owner's accumulator acc (then the result replaces acc)
        auto hop_into_v = [&](float (&v)[16], const Vec8& xw, uint32_t& sub, uint32_t event) {
            char* entry = fifo + (hops++ & 1u) * kFifoEntryBytes;
            chain_send<LPB, RS>(v, entry, QRS ? trace_of(event) : nullptr, lane, sub, active, a.neg_zero);
            widen_bf16x16(xw, v);
            chain_receive<LPB, RS>(v, entry, sub, active);
        };
        auto hop_into_acc = [&](const float (&v)[16], float (&acc)[16], uint32_t& sub, uint32_t event) {
            char* entry = fifo + (hops++ & 1u) * kFifoEntryBytes;
            chain_send<LPB, RS>(v, entry, QRS ? trace_of(event) : nullptr, lane, sub, active, a.neg_zero);
            chain_receive<LPB, RS>(acc, entry, sub, active);
        };

        float acc[16];                     // the owner's reduced tile
        uint32_t sub;                      // this lane's position in the tile
        if (!SEMI) {
            sub = lane;
            {
                const Vec8 x0 = fetch(k + 1, sub);
                widen_bf16x16(x0, acc);
            }
            for (uint32_t j = 1; j < N; ++j) {                                   // hop into rank k+1+j
                const Vec8 xw = fetch(k + 1 + j, sub ^ 1u);
                hop_into_v(acc, xw, sub, j - 1);
            }
        } else {
            // chain B: k+h+1 -> ... -> k+N-1 -> owner (h-1 hops); starts at position `lane`
            sub = lane;
            const uint32_t acc_pos = h >= 2 ? lane ^ ((h - 1) & 1u) : lane;      // position after B's hops
            {
                const Vec8 xo = fetch(k, acc_pos);
                widen_bf16x16(xo, acc);
            }
            float v[16];
            if (h >= 2) {
                {
                    const Vec8 x0 = fetch(k + h + 1, sub);
                    widen_bf16x16(x0, v);
                }
                for (uint32_t j = 1; j < h; ++j) {
                    if (j + 1 < h) {
                        const Vec8 xw = fetch(k + h + 1 + j, sub ^ 1u);
                        hop_into_v(v, xw, sub, h + j - 1);
                    } else {
                        hop_into_acc(v, acc, sub, h + j - 1);
                    }
                }
            }
            // chain A: k+h -> k+h-1 -> ... -> k+1 -> owner (h hops); starts so that it ends on acc's position
            sub = acc_pos ^ (h & 1u);
            {
                const Vec8 x0 = fetch(k + h, sub);
                widen_bf16x16(x0, v);
            }
            for (uint32_t j = 1; j <= h; ++j) {
                if (j < h) {
                    const Vec8 xw = fetch(k + h - j, sub ^ 1u);
                    hop_into_v(v, xw, sub, j - 1);
                } else {
                    hop_into_acc(v, acc, sub, j - 1);
                }
            }
        }

        // all-gather: one more message, quantized or bf16, dequantized/forwarded to every rank
        Vec8 o = {};
        {
            constexpr int AG = QAG ? PAYLOAD : 0;
            char* entry = fifo + (hops++ & 1u) * kFifoEntryBytes;
            chain_send<LPB, AG>(acc, entry, QAG ? trace_of(N - 1) : nullptr, lane, sub, active, a.neg_zero);
            if (QAG) {
                uint4 c = make_uint4(0, 0, 0, 0);
                float s = 0.0f;
                if (active) {
                    c = ld_coherent_128(entry + kRecordHeader + sub * 16);
                    s = ld_coherent_f32(reinterpret_cast<const float*>(entry) + sub / LPB);
                }
                o = dequant_to_bf16_payload<PAYLOAD>(c, s);
            } else if (active) {
                o = ld_fifo_256(entry + sub * 32);
            }
        }
        if (active) {
            const uint64_t byte_off = (tile_off + sub * 16) * 2;
            for (uint32_t r = 0; r < N; ++r) st_stream_256(static_cast<char*>(a.out[r]) + byte_off, o);
        }
        __syncwarp();                      // the next tile reuses the FIFO
    }
}

// The same flavours with every message kept in registers (used when no trace is asked for): the
// lane that produced a group's message goes on as the receiving rank, as in chain_fused_kernel.
// One hop: the message of v (quantized with the flavour's payload, or rounded to bf16) is folded
// into `addend` by the receiver; `out` may be v or addend.
template <int LPB, int PAYLOAD>
__device__ __forceinline__ void fused_hop(const float (&v)[16], const float (&addend)[16], float (&out)[16],
                                          float neg_zero) {
    if (PAYLOAD == 1) {
        float q[16], scale;
        quantize_lane_values<LPB>(v, q, scale, neg_zero);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            fma2_rn(out[2 * i], out[2 * i + 1], q[2 * i], q[2 * i + 1], scale, addend[2 * i], addend[2 * i + 1]);
    } else if (PAYLOAD != 0) {
        uint4 codes;
        float q[16], scale;
        quantize_lane_payload<LPB, PAYLOAD == 0 ? 2 : PAYLOAD>(v, codes, scale, neg_zero);
        decode_x16<PAYLOAD == 0 ? 2 : PAYLOAD>(codes, q);
#pragma unroll
        for (int i = 0; i < 8; ++i)
            fma2_rn(out[2 * i], out[2 * i + 1], q[2 * i], q[2 * i + 1], scale, addend[2 * i], addend[2 * i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t m = pack_bf16x2_rn(v[2 * i], v[2 * i + 1]);                  // the bf16 message
            const uint32_t sum = pack_bf16x2_rn(__fadd_rn(__uint_as_float(m << 16), addend[2 * i]),
                                                __fadd_rn(__uint_as_float(m & 0xFFFF0000u), addend[2 * i + 1]));
            out[2 * i] = __uint_as_float(sum << 16);
            out[2 * i + 1] = __uint_as_float(sum & 0xFFFF0000u);
        }
    }
}

template <int LPB, bool SEMI, bool QRS, bool QAG, int PAYLOAD>
__global__ void __launch_bounds__(kPipeThreads) flavour_fused_kernel(const __grid_constant__ FlavourArgs a) {
    constexpr int RS = QRS ? PAYLOAD : 0;
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps = (uint64_t)gridDim.x * (kPipeThreads / 32);
    const uint64_t warp = (uint64_t)blockIdx.x * (kPipeThreads / 32) + (threadIdx.x >> 5);
    const uint32_t N = a.nranks;
    const uint32_t h = N / 2;
    const uint64_t groups = a.shard >> 4;
    const uint64_t tiles = a.tiles_per_shard * N;

    for (uint64_t tile = warp; tile < tiles; tile += warps) {
        const uint32_t k = (uint32_t)(tile / a.tiles_per_shard);
        const uint64_t t = tile - (uint64_t)k * a.tiles_per_shard;
        const bool active = t * 32 + lane < groups;
        const uint64_t off = ((uint64_t)k * a.shard + (t * 32 + lane) * 16) * 2;    // this lane's group, in bytes
        auto fetch = [&](uint32_t rank) {
            Vec8 x = {};
            if (active) x = ld_coherent_256(static_cast<const char*>(a.in[rank % N]) + off);
            return x;
        };
        // a chain: v starts as rank `first`'s shard and hops through `hops` further ranks (rank first + dir * j)
        auto run_chain = [&](float (&v)[16], uint32_t first, int dir, uint32_t hops) {
            {
                const Vec8 x0 = fetch(first);
                widen_bf16x16(x0, v);
            }
            if (hops == 0) return;
            Vec8 nx = fetch(first + N + dir);
            for (uint32_t j = 1; j <= hops; ++j) {
                float x[16];
                widen_bf16x16(nx, x);
                if (j < hops) nx = fetch(first + N * (j + 1) + dir * (int)(j + 1));   // next counterpart, in flight
                fused_hop<LPB, RS>(v, x, v, a.neg_zero);
            }
        };

        float acc[16];                     // the owner's reduced group
        if (!SEMI) {
            run_chain(acc, k + 1, +1, N - 1);                       // k+1 -> k+2 -> ... -> k
        } else {
            {
                const Vec8 xo = fetch(k);
                widen_bf16x16(xo, acc);
            }
            float v[16];
            if (h >= 2) {                                           // chain B: k+h+1 -> ... -> k+N-1 -> owner
                run_chain(v, k + h + 1, +1, h - 2);
                fused_hop<LPB, RS>(v, acc, acc, a.neg_zero);
            }
            run_chain(v, k + h, -1, h - 1);                         // chain A: k+h -> ... -> k+1 -> owner
            fused_hop<LPB, RS>(v, acc, acc, a.neg_zero);
        }

        // all-gather: one more quantize/dequantize pair, or the sum rounded to bf16
        Vec8 o;
        if (QAG && PAYLOAD == 1) {
            float q[16], scale;
            quantize_lane_values<LPB>(acc, q, scale, a.neg_zero);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float lo, hi;
                mul2_rn(lo, hi, q[2 * i], q[2 * i + 1], scale);
                o.w[i] = pack_bf16x2_rn(lo, hi);
            }
        } else if (QAG) {
            uint4 codes;
            float scale;
            quantize_lane_payload<LPB, PAYLOAD>(acc, codes, scale, a.neg_zero);
            o = dequant_to_bf16_payload<PAYLOAD>(codes, scale);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) o.w[i] = pack_bf16x2_rn(acc[2 * i], acc[2 * i + 1]);
        }
        if (active)
            for (uint32_t r = 0; r < N; ++r) st_stream_256(static_cast<char*>(a.out[r]) + off, o);
    }
}

// ---------------------------------------------------------------- the ring across devices
// The paper's own setting (Section 3, Fig. 1; Section 3.1, Fig. 2): one rank per device, every
// reduce-scatter step a send to the right neighbour and a receive from the left one, metadata
// ahead of the payload, microshards pipelined.  A rank's kernel is ONE persistent launch that runs
// all N ring steps and the all-gather; a microshard is a 512-element tile, its message one
// 544-byte record.  The sender stores the record straight into the RECEIVER's mailbox (plain
// 16-byte stores: over NVLink when the mailbox lives on another GPU) and then, behind a system-scope
// fence, sets a per-tile flag word; the receiver's warp for that tile polls the flag with a BOUNDED
// wait (acquire loads).  Tiles advance
// independently, so a tile's hop overlaps the transfers of all other tiles.  The last
// reduce-scatter step stores the all-gather message of the rank's own shard into every rank's
// mailbox (each peer is reachable at full bandwidth through the switch), and every rank
// dequantizes what it received.  Only plain loads and stores touch peer memory: no bulk-tensor copy, no one-to-many load.
//
// Mailbox of a rank (device memory, zeroed once before its first use):
//   slots 0..N-2   : the message received at ring step s = slot + 1 (tiles_per_shard records)
//   slots N-1..2N-2: the all-gather message of shard k = slot - (N-1)
//   then one 32-bit flag per (slot, tile); a flag equal to the call's epoch means "record complete".
// Epochs grow from call to call, so nothing is cleared between calls.  A slot is only rewritten
// after its reader is done with it: rank r's call e returns only once it holds the all-gather
// record of every tile of every shard, and rank q produces tile t of its all-gather message after
// its last read of tile t of any reduce-scatter slot (one warp owns a tile index through all steps).
//
// A launch can host several consecutive ranks (ranks_here > 1): their CTAs are co-resident (the
// launch is cooperative) and exchange through the same mailboxes, which is how the whole ring runs
// and is checked on a single GPU.
constexpr int kRingThreads = 128;       // 64 and 256 measured on one GPU: 5-8 % slower
constexpr uint32_t kRingBatch = 8;      // tiles whose records share one system-scope fence (2 / 4 / 8: 920 / 731 / 686 us at 88 MB per rank)

struct RingArgs {
    const void* in[kMaxRanks];       // input tensor of hosted rank rank_first + i
    void* out[kMaxRanks];            // output tensor of hosted rank rank_first + i
    char* mailbox[kMaxRanks];        // mailbox of EVERY rank of the ring, as addressable from this device
    uint32_t* status;                // {epoch of the failed call, rank, step, tile}: first failure of this launch, else untouched
    uint64_t shard;
    uint64_t tiles_per_shard;
    uint64_t timeout_ns;             // longest wait for one message
    uint32_t nranks, rank_first, ranks_here, ctas_per_rank;
    uint32_t epoch;
    float neg_zero;
};

__device__ __forceinline__ uint32_t ld_acquire_sys_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_sys_u32(uint32_t* p, uint32_t v) {
    asm volatile("st.relaxed.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_sys() {
    asm volatile("fence.acq_rel.sys;" ::: "memory");
}
// data written by another device (or another SM): strong loads, never served from a stale L1 line
__device__ __forceinline__ uint4 ld_relaxed_sys_128(const void* p) {
    uint4 r;
    asm volatile("ld.relaxed.sys.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ float ld_relaxed_sys_f32(const float* p) {
    float r;
    asm volatile("ld.relaxed.sys.global.f32 %0, [%1];" : "=f"(r) : "l"(p) : "memory");
    return r;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Lane 0 polls the flag until it holds `epoch` or the time limit passes; the verdict is
// broadcast, and the acquire orders the record loads of every lane after the flag.
// A wait also gives up as soon as another warp of this launch has recorded a failure.
__device__ __forceinline__ bool ring_wait(const uint32_t* flag, uint32_t epoch, uint64_t timeout_ns,
                                          const uint32_t* status, uint32_t lane) {
    uint32_t ok = 1;
    if (lane == 0) {
        if (ld_acquire_sys_u32(flag) != epoch) {
            const uint64_t t0 = global_timer_ns();
            for (uint32_t spins = 1;; ++spins) {
                if (ld_acquire_sys_u32(flag) == epoch) break;
                if ((spins & 15u) == 0 &&
                    (global_timer_ns() - t0 > timeout_ns || *reinterpret_cast<const volatile uint32_t*>(status) == epoch)) {
                    ok = 0;
                    break;
                }
                __nanosleep(64);
            }
        }
    }
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    __syncwarp();                    // orders the other lanes' record loads after lane 0's acquire
    return ok != 0;
}

template <int LPB>
__global__ void __launch_bounds__(kRingThreads) ring_rank_kernel(const __grid_constant__ RingArgs a) {
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t N = a.nranks;
    const uint32_t local = blockIdx.x / a.ctas_per_rank;             // hosted rank index
    const uint32_t r = a.rank_first + local;                          // this CTA's rank
    const uint32_t right = r + 1 == N ? 0 : r + 1;
    const uint64_t warps = (uint64_t)a.ctas_per_rank * (kRingThreads / 32);
    const uint64_t warp = (uint64_t)(blockIdx.x - local * a.ctas_per_rank) * (kRingThreads / 32) + (threadIdx.x >> 5);
    const uint64_t T = a.tiles_per_shard;
    const uint64_t groups = a.shard >> 4;
    const uint64_t slot_bytes = T * kRecordBytes;
    const uint64_t flags_at = (uint64_t)(2 * N - 1) * slot_bytes;     // byte offset of the flag words
    const char* const x_rank = static_cast<const char*>(a.in[local]);
    char* const my_box = a.mailbox[r];
    auto flag_of = [&](char* box, uint32_t slot, uint64_t t) {
        return reinterpret_cast<uint32_t*>(box + flags_at) + (uint64_t)slot * T + t;
    };
    // a failing call stamps the status with its own epoch (first failure wins); then this warp leaves
    auto fail = [&](uint32_t step, uint64_t t) {
        if (lane == 0) {
            const uint32_t seen = *reinterpret_cast<volatile uint32_t*>(a.status);
            if (seen != a.epoch && atomicCAS(a.status, seen, a.epoch) == seen) {
                a.status[1] = r;
                a.status[2] = step;
                a.status[3] = (uint32_t)t;
            }
        }
    };

    // ---- reduce-scatter: step s sends shard (r - 1 - s) mod N
    // A warp sends its tiles in batches of up to kRingBatch: the records of a batch are stored, ONE
    // system-scope fence orders them, then the batch's flags are stored.  A fence across NVLink costs
    // microseconds; the batch shares it.  A tile of step s waits only for tiles of step s - 1, so
    // holding a flag back until its batch is complete cannot make a cycle of waits.
    for (uint32_t s = 0; s < N; ++s) {
        const uint32_t k = (r + 2 * N - 1 - s) % N;
        const bool last = s + 1 == N;                                 // k == r: the shard is reduced
        for (uint64_t t0 = warp; t0 < T; t0 += warps * kRingBatch) {
            uint32_t sent = 0;
            for (uint64_t t = t0; sent < kRingBatch && t < T; t += warps, ++sent) {
                const bool active = t * 32 + lane < groups;
                Vec8 xw = {};
                if (active) xw = ld_coherent_256(x_rank + ((uint64_t)k * a.shard + (t * 32 + lane) * 16) * 2);   // in place is allowed
                float v[16];
                widen_bf16x16(xw, v);
                if (s > 0) {                                          // the message received at this step
                    if (!ring_wait(flag_of(my_box, s - 1, t), a.epoch, a.timeout_ns, a.status, lane)) {
                        fail(s, t);
                        return;
                    }
                    const char* rec = my_box + (uint64_t)(s - 1) * slot_bytes + t * kRecordBytes;
                    uint4 c = make_uint4(0, 0, 0, 0);
                    float sc = 0.0f;
                    if (active) {
                        c = ld_relaxed_sys_128(rec + kRecordHeader + lane * 16);
                        sc = ld_relaxed_sys_f32(reinterpret_cast<const float*>(rec) + lane / LPB);
                    }
                    dequant_add_x16(c, sc, v);
                }
                uint4 codes;
                float scale;
                quantize_lane<LPB>(v, codes, scale, a.neg_zero);
                float hdr = __shfl_sync(0xFFFFFFFFu, scale, (lane * LPB) & 31u);   // lanes 0..7: the metadata sector
                if (lane >= 32u / LPB) hdr = 0.0f;
                // to the right neighbour, as the message it receives at step s + 1; the reduced shard's
                // all-gather message goes to every rank
                const uint32_t slot = last ? N - 1 + k : s;
                for (uint32_t q = last ? 0 : right; q < (last ? N : right + 1); ++q) {
                    char* rec = a.mailbox[q] + (uint64_t)slot * slot_bytes + t * kRecordBytes;
                    if (lane < 8) st_plain_f32(reinterpret_cast<float*>(rec) + lane, hdr);
                    if (active) st_plain_128(rec + kRecordHeader + lane * 16, codes);
                }
            }
            __syncwarp();                                             // every lane's stores happen before lane 0's fence
            if (lane == 0) {
                fence_acq_rel_sys();
                const uint32_t slot = last ? N - 1 + k : s;
                uint64_t t = t0;
                for (uint32_t i = 0; i < sent; ++i, t += warps)
                    for (uint32_t q = last ? 0 : right; q < (last ? N : right + 1); ++q)
                        st_relaxed_sys_u32(flag_of(a.mailbox[q], slot, t), a.epoch);
            }
        }
    }

    // ---- all-gather receive side: dequantize every shard's message into this rank's output
    char* const out_rank = static_cast<char*>(a.out[local]);
    for (uint32_t i = 0; i < N; ++i) {
        const uint32_t k = (r + i) % N;                               // own shard first: it is already here
        for (uint64_t t = warp; t < T; t += warps) {
            if (!ring_wait(flag_of(my_box, N - 1 + k, t), a.epoch, a.timeout_ns, a.status, lane)) {
                fail(N + k, t);
                return;
            }
            if (t * 32 + lane >= groups) continue;
            const char* rec = my_box + (uint64_t)(N - 1 + k) * slot_bytes + t * kRecordBytes;
            const uint4 c = ld_relaxed_sys_128(rec + kRecordHeader + lane * 16);
            const float sc = ld_relaxed_sys_f32(reinterpret_cast<const float*>(rec) + lane / LPB);
            const Vec8 o = dequant_to_bf16x16(c, sc);
            st_stream_256(out_rank + ((uint64_t)k * a.shard + (t * 32 + lane) * 16) * 2, o);
        }
    }
}

// Unquantized comparator hop: send = bf16_rne(f32(recv) + f32(local)).
__global__ void __launch_bounds__(kThreads) bf16_step_kernel(const __grid_constant__ Bf16StepArgs a) {
    const uint32_t r = blockIdx.y;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool active = g < (a.shard >> 4);
    Vec8 lw = {};
    if (active) lw = ld_stream_256(static_cast<const char*>(a.local[r]) + g * 32);
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    if (!active) return;
    // the received shard was written by the previous launch (or is a neighbour's input)
    Vec8 rw;
    {
        const uint4* p = reinterpret_cast<const uint4*>(static_cast<const char*>(a.recv[r]) + g * 32);
        const uint4 lo = __ldcg(p), hi = __ldcg(p + 1);
        rw.w[0] = lo.x; rw.w[1] = lo.y; rw.w[2] = lo.z; rw.w[3] = lo.w;
        rw.w[4] = hi.x; rw.w[5] = hi.y; rw.w[6] = hi.z; rw.w[7] = hi.w;
    }
    float x[16], y[16];
    widen_bf16x16(lw, x);
    widen_bf16x16(rw, y);
    Vec8 o;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        o.w[i] = pack_bf16x2_rn(__fadd_rn(y[2 * i], x[2 * i]), __fadd_rn(y[2 * i + 1], x[2 * i + 1]));
    uint4* q = reinterpret_cast<uint4*>(static_cast<char*>(a.send[r]) + g * 32);
    __stcg(q, make_uint4(o.w[0], o.w[1], o.w[2], o.w[3]));
    __stcg(q + 1, make_uint4(o.w[4], o.w[5], o.w[6], o.w[7]));
}

// Unquantized all-gather: copy reduced shard k into every output.
__global__ void __launch_bounds__(kThreads) bf16_gather_kernel(const __grid_constant__ Bf16GatherArgs a) {
    const uint32_t k = blockIdx.y;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    if (g >= (a.shard >> 4)) return;
    const uint4* p = reinterpret_cast<const uint4*>(static_cast<const char*>(a.src[k]) + g * 32);
    const uint4 lo = __ldcg(p), hi = __ldcg(p + 1);
    Vec8 o;
    o.w[0] = lo.x; o.w[1] = lo.y; o.w[2] = lo.z; o.w[3] = lo.w;
    o.w[4] = hi.x; o.w[5] = hi.y; o.w[6] = hi.z; o.w[7] = hi.w;
    const uint64_t byte_off = (k * a.shard + g * 16) * 2;
    for (uint32_t r = 0; r < a.nranks; ++r) st_stream_256(static_cast<char*>(a.out[r]) + byte_off, o);
}

}  // namespace equarx
