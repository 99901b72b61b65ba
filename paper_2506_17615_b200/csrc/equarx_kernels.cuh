// sm_100a kernels for the EQuARX hot path: block-wise int8 quantize, the fused
// dequantize / fp32 add / requantize of a ring hop, and the all-gather
// dequantize (arXiv 2506.17615, Sections 3.1, 3.2, 3.4).
//
// Thread mapping, shared by every kernel: one lane owns 16 contiguous
// elements (one 256-bit bf16 access, one 128-bit int8 access), so a block of
// B elements is B/16 neighbouring lanes of one warp and the per-block max is
// an in-lane max followed by log2(B/16) shuffles.  grid.y is the simulated
// rank (or, in the all-gather, the shard); grid.x tiles the shard.
//
// Every floating-point step that decides a bit of the result uses an explicit
// round-to-nearest intrinsic, so the compiler cannot contract or reorder it:
//   scale = __fdiv_rn(amax, 127), inv = __fdiv_rn(127, amax)
//   code  = rne(__fmul_rn(v, inv))    (the add of 1.5*2^23 rounds to the integer grid)
//   hop   = __fmaf_rn((float)code, scale, local)
//   final = cvt.rn.bf16(__fmul_rn((float)code, scale))
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace equarx {

constexpr int kThreads = 256;        // threads per CTA
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
__device__ __forceinline__ uint64_t policy_keep() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}

__device__ __forceinline__ uint4 ld_wire_128(const void* p, uint64_t pol) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.b32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                 : "l"(p), "l"(pol));
    return r;
}

__device__ __forceinline__ void st_wire_128(void* p, const uint4& r, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1,%2,%3,%4}, %5;"
                 ::"l"(p), "r"(r.x), "r"(r.y), "r"(r.z), "r"(r.w), "l"(pol)
                 : "memory");
}

__device__ __forceinline__ float ld_scale(const float* p, uint64_t pol) {
    float r;
    asm volatile("ld.global.nc.L2::cache_hint.f32 %0, [%1], %2;" : "=f"(r) : "l"(p), "l"(pol));
    return r;
}

__device__ __forceinline__ void st_scale(float* p, float v, uint64_t pol) {
    asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(v), "l"(pol) : "memory");
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
        q[4 * j + 0] = __fsub_rn(__uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7540)), 8388736.0f);
        q[4 * j + 1] = __fsub_rn(__uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7541)), 8388736.0f);
        q[4 * j + 2] = __fsub_rn(__uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7542)), 8388736.0f);
        q[4 * j + 3] = __fsub_rn(__uint_as_float(__byte_perm(w[j], 0x4B000000u, 0x7543)), 8388736.0f);
    }
}

template <int LPB>
__device__ __forceinline__ float block_max(float m) {
#pragma unroll
    for (int off = LPB / 2; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
    return m;
}

// Q_p1 + Q_p2 on the 16 values of one lane; the block is LPB neighbouring lanes.
// |v * inv| <= 127 * (1 + 2^-24)^2 < 127.5, so the rounded code never leaves
// [-127, 127] and needs no clamp; adding 1.5 * 2^23 rounds to nearest-even on the
// integer grid and leaves the two's-complement code in the low byte.
template <int LPB>
__device__ __forceinline__ void quantize_lane(const float (&v)[16], uint4& codes, float& scale) {
    float m = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) m = fmaxf(m, fabsf(v[i]));
    m = block_max<LPB>(m);
    float inv;
    if (m >= 0x1p-118f) {
        scale = __fdiv_rn(m, 127.0f);
        inv = __fdiv_rn(127.0f, m);
    } else {
        scale = 0.0f;
        inv = 0.0f;
    }
    uint32_t b[16];
#pragma unroll
    for (int i = 0; i < 16; ++i)
        b[i] = __float_as_uint(__fadd_rn(__fmul_rn(v[i], inv), 12582912.0f));
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t lo = __byte_perm(b[4 * j + 0], b[4 * j + 1], 0x0040);
        const uint32_t hi = __byte_perm(b[4 * j + 2], b[4 * j + 3], 0x0040);
        o[j] = __byte_perm(lo, hi, 0x5410);
    }
    codes = make_uint4(o[0], o[1], o[2], o[3]);
}

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// ---------------------------------------------------------------- kernel arguments
// One launch covers every simulated rank.  Messages live in "slots" of a scales
// region and a codes region (slot * bps floats, slot * shard bytes).
struct StepArgs {
    const void* x[kMaxRanks];        // rank r's bf16 shard for this step
    uint32_t in_slot[kMaxRanks];     // message received by rank r (unused at step 0)
    uint32_t out_slot[kMaxRanks];    // message produced by rank r
    const int8_t* codes_in;
    const float* scales_in;
    int8_t* codes_out;
    float* scales_out;
    uint64_t shard;                  // elements per message
    uint64_t bps;                    // blocks per message
};

struct GatherArgs {
    void* out[kMaxRanks];            // output tensor of rank r (whole tensor)
    uint32_t slot[kMaxRanks];        // final message of shard k
    const int8_t* codes;
    const float* scales;
    uint64_t shard;
    uint64_t bps;
    uint32_t nranks;
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
// Step 0 is never launched as a programmatic dependent: it reads tensors that an
// earlier in-place all-gather on the same stream may still be writing.
template <int LPB, bool FIRST>
__global__ void __launch_bounds__(kThreads) rs_step_kernel(const __grid_constant__ StepArgs a) {
    const uint32_t r = blockIdx.y;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;   // 16-element group
    const bool active = g < (a.shard >> 4);
    const uint64_t pol = policy_keep();

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
            c = ld_wire_128(a.codes_in + slot * a.shard + g * 16, pol);
            s = ld_scale(a.scales_in + slot * a.bps + g / LPB, pol);
        }
        float q[16];
        codes_to_f32x16(c, q);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = __fmaf_rn(q[i], s, v[i]);
    }

    uint4 codes;
    float scale;
    quantize_lane<LPB>(v, codes, scale);
    if (active) {
        const uint64_t slot = a.out_slot[r];
        st_wire_128(a.codes_out + slot * a.shard + g * 16, codes, pol);
        if ((threadIdx.x & (LPB - 1)) == 0) st_scale(a.scales_out + slot * a.bps + g / LPB, scale, pol);
    }
}

// All-gather receive side: one read of shard k's final message, nranks bf16 writes.
template <int LPB>
__global__ void __launch_bounds__(kThreads) ag_dequant_kernel(const __grid_constant__ GatherArgs a) {
    const uint32_t k = blockIdx.y;
    const uint64_t g = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool active = g < (a.shard >> 4);
    const uint64_t pol = policy_keep();
    pdl_launch_dependents();
    pdl_wait_prior_grid();
    if (!active) return;
    const uint64_t slot = a.slot[k];
    const uint4 c = ld_wire_128(a.codes + slot * a.shard + g * 16, pol);
    const float s = ld_scale(a.scales + slot * a.bps + g / LPB, pol);
    float q[16];
    codes_to_f32x16(c, q);
    Vec8 o;
#pragma unroll
    for (int i = 0; i < 8; ++i)
        o.w[i] = pack_bf16x2_rn(__fmul_rn(q[2 * i], s), __fmul_rn(q[2 * i + 1], s));
    const uint64_t byte_off = (k * a.shard + g * 16) * 2;
    for (uint32_t r = 0; r < a.nranks; ++r) st_stream_256(static_cast<char*>(a.out[r]) + byte_off, o);
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
