/*
 * EQuARX CPU oracle -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, single-threaded restatement of the arithmetic that EQuARX
 * (arXiv 2506.17615) runs beside the steps of a ring AllReduce: dynamic
 * block-wise int8 quantization (Section 3.2), the dequantize -> fp32 add ->
 * requantize of every reduce-scatter hop (Section 3.1), and the extra
 * quantize/dequantize pair of the quantized all-gather (Section 3.4), in the
 * fixed order of the full-loop ring (Section 3, Fig. 1; Section 3.3, Fig. 4).
 *
 * Only the tests, the smoke check and the bench's cpu_baseline / reference
 * legs may call this file.  It shares no code, header, table or constant
 * with the CUDA library; the CUDA library never calls it.
 *
 * The method is an approximation with a fixed evaluation order, so this file
 * takes the algorithm step by step in the paper's order (ring step 0 sends a
 * quantized shard; every later step dequantizes the received shard to fp32,
 * adds the local counterpart, requantizes and forwards; the all-gather
 * forwards the last message and everybody dequantizes it).  There is no
 * blocking, fusion or reordering beyond that.  Precision is the paper's:
 * bf16 tensors, int8 payload, fp32 accumulation (Section 3.1 widens the
 * received shard before adding and names FP32).  Where the paper is silent the reading taken is
 * stated next to the code:
 *   - ring direction: rank r sends to rank (r+1) mod N; shard k ends on
 *     rank k (the semi-loop example of Section 3.3 finishes shard 0 on
 *     device 0).
 *   - a block is B contiguous elements of a shard with one fp32 scale
 *     (Fig. 3 caption: one scale per block of entries; the 8x128 strided
 *     layout of Section 3.2 is a TPU register artefact and is not used).
 *   - symmetric quantization to [-127, 127]: scale = amax / 127 (the
 *     dequantization multiplier, which is what travels as metadata),
 *     code = clamp(rne(v * (127 / amax))), both divisions IEEE fp32.
 *   - blocks with amax < 2^-118 (zero blocks included) get scale 0 and all
 *     codes 0, so that the scale is never subnormal and nothing depends on
 *     flush-to-zero behaviour.
 *   - dequantize-and-add is one fused multiply-add fmaf(code, scale, local).
 *   - the partial sum stays fp32 between the add and the requantization.
 *   - every rank, the owner included, outputs bf16_rne(code * scale) of the
 *     all-gather message, so all N outputs are bit-identical.
 *   - Inf/NaN inputs are outside the contract (status 9).
 *
 * Pins (tests/test_oracle_*.py): hand-worked blocks, tie and range blocks,
 * exact-integer reductions that must equal a plain integer sum, an exact
 * rational re-evaluation on tiny inputs, scaling / negation / permutation /
 * rotation invariants, the a-posteriori error bound against the fp64 sum,
 * and the mean squared errors printed in Section 4.1 (Fig. 7).
 * Unpinned (declared choices, nothing in the paper or mathematics fixes
 * them): the ring direction and the 2^-118 flush threshold.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fPIC -shared (no -ffast-math).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum {
    ORACLE_OK = 0,
    ORACLE_ERR_NULL = 1,
    ORACLE_ERR_NRANKS = 2,
    ORACLE_ERR_BLOCK = 3,
    ORACLE_ERR_COUNT = 4,
    ORACLE_ERR_ALLOC = 6,
    ORACLE_ERR_NONFINITE = 9
};

/* bf16 <-> fp32.  bf16 is the upper half of an fp32 word, so widening is exact. */
static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* fp32 -> bf16, round to nearest, ties to even (finite input). */
static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    uint32_t keep_lsb = (u >> 16) & 1u;
    u += 0x7FFFu + keep_lsb;
    return (uint16_t)(u >> 16);
}

static int bf16_is_finite(uint16_t h) { return (h & 0x7F80u) != 0x7F80u; }

/*
 * Q_p1 + Q_p2 of Section 3.1 on one block of `block` fp32 values:
 * first pass finds the metadata (max |v|), second pass scales the data.
 */
static void quantize_one_block(const float *v, int block, int8_t *code, float *scale_out)
{
    float amax = 0.0f;
    for (int i = 0; i < block; ++i) {
        float a = fabsf(v[i]);
        if (a > amax) amax = a;
    }
    float scale, inv;
    if (!(amax >= 0x1p-118f)) {
        scale = 0.0f;
        inv = 0.0f;
    } else {
        scale = amax / 127.0f;
        inv = 127.0f / amax;
    }
    for (int i = 0; i < block; ++i) {
        float t = v[i] * inv;
        float r = rintf(t);          /* default rounding mode: ties to even */
        if (r > 127.0f) r = 127.0f;
        if (r < -127.0f) r = -127.0f;
        code[i] = (int8_t)r;
    }
    *scale_out = scale;
}

/*
 * FP8 payloads (Section 4: "int8, FP8 (E4M3) and FP8 (E5M2), and it uses symmetric
 * quantization").  Reading: the same block-wise rule with the format's largest finite
 * value in place of 127: scale = amax / FMAX, code = fp8_rne(v * (FMAX / amax)),
 * saturating at +-FMAX; E4M3 is the 8-bit format with bias 7, no infinities and
 * FMAX = 448, E5M2 the one with bias 15 and FMAX = 57344.  Blocks with
 * amax < FMAX_pow2 * 2^-126 (2^-117 for E4M3, 2^-110 for E5M2) get scale 0 and zero
 * codes, which keeps the scale normal and FMAX / amax finite.
 */
typedef struct { int p; int emin; int bias; float fmax; float flush; } fp8_format;
static const fp8_format FP8_E4M3 = {4, -6, 7, 448.0f, 0x1p-117f};
static const fp8_format FP8_E5M2 = {3, -14, 15, 57344.0f, 0x1p-110f};

/* round t to the nearest value of the format (ties to even), saturating at +-fmax */
static float fp8_round(float t, const fp8_format *f)
{
    if (t == 0.0f) return t;
    float a = fabsf(t);
    int e;
    (void)frexpf(a, &e);                 /* a = m * 2^e, m in [0.5, 1): floor(log2 a) = e - 1 */
    int E = e - 1;
    if (E < f->emin) E = f->emin;        /* subnormals share the spacing of emin */
    float ulp = ldexpf(1.0f, E - (f->p - 1));
    float r = rintf(a / ulp) * ulp;      /* both scalings are by powers of two: exact */
    if (r > f->fmax) r = f->fmax;
    return copysignf(r, t);
}

/* the byte that encodes a value of the format: sign, exponent field, p-1 mantissa bits */
static uint8_t fp8_encode(float r, const fp8_format *f)
{
    uint8_t sign = signbit(r) ? 0x80u : 0u;
    float a = fabsf(r);
    if (a == 0.0f) return sign;
    int e;
    (void)frexpf(a, &e);
    int E = e - 1;
    unsigned field, mant;
    if (E < f->emin) {
        field = 0;
        mant = (unsigned)(a / ldexpf(1.0f, f->emin - (f->p - 1)));
    } else {
        field = (unsigned)(E + f->bias);
        mant = (unsigned)((a / ldexpf(1.0f, E) - 1.0f) * (float)(1 << (f->p - 1)));
    }
    return (uint8_t)(sign | (field << (f->p - 1)) | mant);
}

static float fp8_decode(uint8_t byte, const fp8_format *f)
{
    unsigned field = (byte & 0x7Fu) >> (f->p - 1);
    unsigned mant = byte & ((1u << (f->p - 1)) - 1u);
    float a = field == 0 ? (float)mant * ldexpf(1.0f, f->emin - (f->p - 1))
                         : (1.0f + (float)mant / (float)(1 << (f->p - 1))) * ldexpf(1.0f, (int)field - f->bias);
    return (byte & 0x80u) ? -a : a;
}

/* payload: 0 int8, 1 FP8 E4M3, 2 FP8 E5M2.  Codes are stored as raw bytes. */
static void quantize_one_block_payload(const float *v, int block, int payload, int8_t *code, float *scale_out)
{
    if (payload == 0) {
        quantize_one_block(v, block, code, scale_out);
        return;
    }
    const fp8_format *f = payload == 1 ? &FP8_E4M3 : &FP8_E5M2;
    float amax = 0.0f;
    for (int i = 0; i < block; ++i) {
        float a = fabsf(v[i]);
        if (a > amax) amax = a;
    }
    float scale, inv;
    if (!(amax >= f->flush)) {
        scale = 0.0f;
        inv = 0.0f;
    } else {
        scale = amax / f->fmax;
        inv = f->fmax / amax;
    }
    for (int i = 0; i < block; ++i) code[i] = (int8_t)fp8_encode(fp8_round(v[i] * inv, f), f);
    *scale_out = scale;
}

static float code_value(int8_t code, int payload)
{
    if (payload == 0) return (float)code;
    return fp8_decode((uint8_t)code, payload == 1 ? &FP8_E4M3 : &FP8_E5M2);
}

static int check_block_count(size_t count, int block)
{
    if (block < 1) return ORACLE_ERR_BLOCK;
    if (count == 0 || count % (size_t)block != 0) return ORACLE_ERR_COUNT;
    return ORACLE_OK;
}

/* Ring step 0: quantize a bf16 buffer block by block (Section 3.1, 3.2). */
int equarx_oracle_quantize_blocks(const uint16_t *x, size_t count, int block,
                                  int8_t *codes, float *scales)
{
    if (!x || !codes || !scales) return ORACLE_ERR_NULL;
    int st = check_block_count(count, block);
    if (st) return st;
    float *v = (float *)malloc((size_t)block * sizeof(float));
    if (!v) return ORACLE_ERR_ALLOC;
    for (size_t b = 0; b < count / (size_t)block; ++b) {
        for (int i = 0; i < block; ++i) {
            uint16_t h = x[b * (size_t)block + i];
            if (!bf16_is_finite(h)) { free(v); return ORACLE_ERR_NONFINITE; }
            v[i] = bf16_to_f32(h);
        }
        quantize_one_block(v, block, codes + b * (size_t)block, scales + b);
    }
    free(v);
    return ORACLE_OK;
}

/*
 * Ring steps 1..N-1: dequantize the received shard to fp32, add the local
 * counterpart, requantize (Section 3.1).
 */
int equarx_oracle_rs_step(const int8_t *codes_in, const float *scales_in,
                          const uint16_t *local, size_t count, int block,
                          int8_t *codes_out, float *scales_out)
{
    if (!codes_in || !scales_in || !local || !codes_out || !scales_out) return ORACLE_ERR_NULL;
    int st = check_block_count(count, block);
    if (st) return st;
    float *v = (float *)malloc((size_t)block * sizeof(float));
    if (!v) return ORACLE_ERR_ALLOC;
    for (size_t b = 0; b < count / (size_t)block; ++b) {
        float s = scales_in[b];
        for (int i = 0; i < block; ++i) {
            size_t e = b * (size_t)block + i;
            if (!bf16_is_finite(local[e])) { free(v); return ORACLE_ERR_NONFINITE; }
            v[i] = fmaf((float)codes_in[e], s, bf16_to_f32(local[e]));
        }
        quantize_one_block(v, block, codes_out + b * (size_t)block, scales_out + b);
    }
    free(v);
    return ORACLE_OK;
}

/* All-gather receive side: dequantize the message to bf16 (Section 3.4). */
int equarx_oracle_ag_dequant(const int8_t *codes, const float *scales, size_t count,
                             int block, uint16_t *out)
{
    if (!codes || !scales || !out) return ORACLE_ERR_NULL;
    int st = check_block_count(count, block);
    if (st) return st;
    for (size_t e = 0; e < count; ++e) {
        float d = (float)codes[e] * scales[e / (size_t)block];
        out[e] = f32_to_bf16_rne(d);
    }
    return ORACLE_OK;
}

static int check_sim_args(int nranks, size_t count, int block)
{
    if (nranks < 1 || nranks > 4096) return ORACLE_ERR_NRANKS;
    if (block < 1) return ORACLE_ERR_BLOCK;
    if (count == 0 || count % ((size_t)nranks * (size_t)block) != 0) return ORACLE_ERR_COUNT;
    return ORACLE_OK;
}

/*
 * Full-loop ring reduce-scatter + all-gather, both stages quantized.
 *
 * in[r], out[r]   : nranks host pointers to `count` bf16 words each.
 * trace_scales    : optional, float [nranks shards][nranks events][count/(nranks*block)]
 * trace_codes     : optional, int8  [nranks shards][nranks events][count/nranks]
 *                   event j of shard k is the message sent at ring step j by
 *                   rank (k+1+j) mod N; event N-1 is the all-gather message.
 * exact_sum       : optional, double[count], sum over ranks of the inputs.
 *
 * The loop below is the ring as the paper draws it: at every step every
 * rank produces one message for its neighbour.  Rank r sends shard
 * (r-1-s) mod N at step s.
 */
int equarx_oracle_allreduce(const uint16_t *const *in, uint16_t *const *out,
                            int nranks, size_t count, int block,
                            float *trace_scales, int8_t *trace_codes, double *exact_sum)
{
    if (!in || !out) return ORACLE_ERR_NULL;
    int st = check_sim_args(nranks, count, block);
    if (st) return st;
    const size_t N = (size_t)nranks;
    const size_t shard = count / N;
    const size_t bps = shard / (size_t)block;   /* blocks per shard */
    for (size_t r = 0; r < N; ++r) {
        if (!in[r] || !out[r]) return ORACLE_ERR_NULL;
        for (size_t e = 0; e < count; ++e)
            if (!bf16_is_finite(in[r][e])) return ORACLE_ERR_NONFINITE;
    }

    if (exact_sum) {
        for (size_t e = 0; e < count; ++e) {
            double s = 0.0;
            for (size_t r = 0; r < N; ++r) s += (double)bf16_to_f32(in[r][e]);
            exact_sum[e] = s;
        }
    }

    /* message held by each rank: msg[cur][r] was produced by rank r in the last step */
    int8_t *msg_codes[2];
    float *msg_scales[2];
    float *v = (float *)malloc((size_t)block * sizeof(float));
    for (int p = 0; p < 2; ++p) {
        msg_codes[p] = (int8_t *)malloc(N * shard);
        msg_scales[p] = (float *)malloc(N * bps * sizeof(float));
    }
    if (!v || !msg_codes[0] || !msg_codes[1] || !msg_scales[0] || !msg_scales[1]) {
        free(v);
        for (int p = 0; p < 2; ++p) { free(msg_codes[p]); free(msg_scales[p]); }
        return ORACLE_ERR_ALLOC;
    }

    for (size_t s = 0; s < N; ++s) {            /* ring step */
        const int cur = (int)(s & 1), prev = cur ^ 1;
        for (size_t r = 0; r < N; ++r) {        /* every rank acts in every step */
            const size_t k = (r + N * 2 - 1 - s) % N;      /* shard handled by rank r now */
            const size_t left = (r + N - 1) % N;           /* the neighbour it received from */
            const uint16_t *mine = in[r] + k * shard;
            int8_t *oc = msg_codes[cur] + r * shard;
            float *os = msg_scales[cur] + r * bps;
            for (size_t b = 0; b < bps; ++b) {
                if (s == 0) {
                    for (int i = 0; i < block; ++i)
                        v[i] = bf16_to_f32(mine[b * (size_t)block + i]);
                } else {
                    const int8_t *ic = msg_codes[prev] + left * shard + b * (size_t)block;
                    const float sc = msg_scales[prev][left * bps + b];
                    for (int i = 0; i < block; ++i)
                        v[i] = fmaf((float)ic[i], sc, bf16_to_f32(mine[b * (size_t)block + i]));
                }
                quantize_one_block(v, block, oc + b * (size_t)block, os + b);
            }
            if (trace_codes)
                memcpy(trace_codes + (k * N + s) * shard, oc, shard);
            if (trace_scales)
                memcpy(trace_scales + (k * N + s) * bps, os, bps * sizeof(float));
        }
    }

    /* all-gather: after step N-1 rank k holds the message of shard k; everybody dequantizes it */
    const int last = (int)((N - 1) & 1);
    for (size_t k = 0; k < N; ++k) {
        const int8_t *c = msg_codes[last] + k * shard;
        const float *sc = msg_scales[last] + k * bps;
        for (size_t e = 0; e < shard; ++e) {
            uint16_t h = f32_to_bf16_rne((float)c[e] * sc[e / (size_t)block]);
            for (size_t r = 0; r < N; ++r) out[r][k * shard + e] = h;
        }
    }

    free(v);
    for (int p = 0; p < 2; ++p) { free(msg_codes[p]); free(msg_scales[p]); }
    return ORACLE_OK;
}

/*
 * The unquantized comparator: the same ring with bf16 messages, fp32 add and
 * a bf16 rounding at every hop ("baseline BF16 AllReduce", Section 4).
 * Step 0 sends the raw shard; the all-gather forwards the reduced shard.
 */
int equarx_oracle_allreduce_bf16(const uint16_t *const *in, uint16_t *const *out,
                                 int nranks, size_t count)
{
    if (!in || !out) return ORACLE_ERR_NULL;
    if (nranks < 1 || nranks > 4096) return ORACLE_ERR_NRANKS;
    if (count == 0 || count % (size_t)nranks != 0) return ORACLE_ERR_COUNT;
    const size_t N = (size_t)nranks;
    const size_t shard = count / N;
    for (size_t r = 0; r < N; ++r) {
        if (!in[r] || !out[r]) return ORACLE_ERR_NULL;
        for (size_t e = 0; e < count; ++e)
            if (!bf16_is_finite(in[r][e])) return ORACLE_ERR_NONFINITE;
    }
    uint16_t *msg[2];
    msg[0] = (uint16_t *)malloc(count * sizeof(uint16_t));
    msg[1] = (uint16_t *)malloc(count * sizeof(uint16_t));
    if (!msg[0] || !msg[1]) { free(msg[0]); free(msg[1]); return ORACLE_ERR_ALLOC; }
    for (size_t s = 0; s < N; ++s) {
        const int cur = (int)(s & 1), prev = cur ^ 1;
        for (size_t r = 0; r < N; ++r) {
            const size_t k = (r + N * 2 - 1 - s) % N;
            const size_t left = (r + N - 1) % N;
            const uint16_t *mine = in[r] + k * shard;
            uint16_t *o = msg[cur] + r * shard;
            for (size_t e = 0; e < shard; ++e) {
                if (s == 0) {
                    o[e] = mine[e];
                } else {
                    float sum = bf16_to_f32(msg[prev][left * shard + e]) + bf16_to_f32(mine[e]);
                    o[e] = f32_to_bf16_rne(sum);
                }
            }
        }
    }
    const int last = (int)((N - 1) & 1);
    for (size_t k = 0; k < N; ++k)
        for (size_t r = 0; r < N; ++r)
            memcpy(out[r] + k * shard, msg[last] + k * shard, shard * sizeof(uint16_t));
    free(msg[0]);
    free(msg[1]);
    return ORACLE_OK;
}

/*
 * The other flavours of Section 3.3 / 3.4, written per shard as the adder chains
 * of Fig. 4 and Fig. 5 (blocks are independent, so the order of shards and
 * blocks is immaterial):
 *
 *   semi_loop = 0: full-loop chain  k+1 -> k+2 -> ... -> k-1 -> k      (N-1 hops)
 *   semi_loop = 1: two half chains that meet at the owner k (N even):
 *                  A: k+N/2 -> k+N/2-1 -> ... -> k+1 -> k              (N/2 hops)
 *                  B: k+N/2+1 -> k+N/2+2 -> ... -> k-1 -> k            (N/2-1 hops)
 *                  (on 4 devices: 2 -> 1 -> 0 and 3 -> 0, the example of Section 3.3);
 *                  B's partial reaches the owner one iteration before A's, so the
 *                  owner adds B's first, then A's.
 *   quant_rs     : hop messages are quantized (else bf16: the add is rounded to
 *                  bf16 at every hop, as in the BF16 baseline);
 *   quant_ag     : the reduced shard goes through one more quantize/dequantize
 *                  pair (else the owner's result is rounded to bf16 and
 *                  forwarded as is).
 * With quant_rs the partial sum stays fp32 from the fused add to the next
 * quantization, also on the semi-loop owner between its two receives.  Without
 * quant_rs the reduce-scatter result is a bf16 tensor, and that is what a
 * quantized all-gather then quantizes.
 *
 * Trace (optional, same shapes as equarx_oracle_allreduce): event j of shard k is
 *   full loop : j = 0..N-2 the hops in chain order, j = N-1 the all-gather message;
 *   semi loop : j = 0..N/2-1 chain A's hops, j = N/2..N-2 chain B's hops, j = N-1
 *               the all-gather message.
 * Events that are not quantized in the chosen flavour are left zero.
 * payload: 0 int8, 1 FP8 E4M3, 2 FP8 E5M2 (codes are the raw bytes).
 */
static void hop_receive(int quant, int payload, const float *v_sent, int block, const float *addend,
                        float *v_out, int8_t *codes, float *scale)
{
    /* sender side: message of v_sent; receiver side: v_out = message (+) addend */
    if (quant) {
        quantize_one_block_payload(v_sent, block, payload, codes, scale);
        for (int i = 0; i < block; ++i) v_out[i] = fmaf(code_value(codes[i], payload), *scale, addend[i]);
    } else {
        for (int i = 0; i < block; ++i) {
            float msg = bf16_to_f32(f32_to_bf16_rne(v_sent[i]));      /* the bf16 message */
            v_out[i] = bf16_to_f32(f32_to_bf16_rne(msg + addend[i])); /* add, rounded to bf16 */
        }
    }
}

int equarx_oracle_allreduce_variant(const uint16_t *const *in, uint16_t *const *out,
                                    int nranks, size_t count, int block,
                                    int semi_loop, int quant_rs, int quant_ag, int payload,
                                    float *trace_scales, int8_t *trace_codes)
{
    if (!in || !out) return ORACLE_ERR_NULL;
    int st = check_sim_args(nranks, count, block);
    if (st) return st;
    if (semi_loop && (nranks % 2 != 0)) return ORACLE_ERR_NRANKS;
    if (payload < 0 || payload > 2) return ORACLE_ERR_BLOCK;
    const size_t N = (size_t)nranks;
    const size_t shard = count / N;
    const size_t bps = shard / (size_t)block;
    for (size_t r = 0; r < N; ++r) {
        if (!in[r] || !out[r]) return ORACLE_ERR_NULL;
        for (size_t e = 0; e < count; ++e)
            if (!bf16_is_finite(in[r][e])) return ORACLE_ERR_NONFINITE;
    }
    if (trace_scales) memset(trace_scales, 0, N * N * bps * sizeof(float));
    if (trace_codes) memset(trace_codes, 0, N * N * shard);

    float *v = (float *)malloc(4 * (size_t)block * sizeof(float));
    int8_t *codes = (int8_t *)malloc((size_t)block);
    if (!v || !codes) { free(v); free(codes); return ORACLE_ERR_ALLOC; }
    float *x = v + block, *acc = v + 2 * (size_t)block, *w = v + 3 * (size_t)block;

    for (size_t k = 0; k < N; ++k) {
        for (size_t b = 0; b < bps; ++b) {
            const size_t base = k * shard + b * (size_t)block;
            size_t event = 0;
            float scale;
#define LOAD(dst, rank) for (int i = 0; i < block; ++i) (dst)[i] = bf16_to_f32(in[(rank) % N][base + (size_t)i])
#define RECORD(quantized) do { if (quantized) { \
                if (trace_scales) trace_scales[(k * N + event) * bps + b] = scale; \
                if (trace_codes) memcpy(trace_codes + (k * N + event) * shard + b * (size_t)block, codes, (size_t)block); } \
                ++event; } while (0)
            if (!semi_loop) {
                LOAD(v, k + 1);
                for (size_t j = 1; j < N; ++j) {           /* hop into rank k+1+j */
                    LOAD(x, k + 1 + j);
                    hop_receive(quant_rs, payload, v, block, x, w, codes, &scale);
                    memcpy(v, w, (size_t)block * sizeof(float));
                    RECORD(quant_rs);
                }
                memcpy(acc, v, (size_t)block * sizeof(float));
            } else {
                const size_t h = N / 2;
                /* chain B first: it reaches the owner one iteration earlier */
                LOAD(acc, k);
                size_t event_b = h;                        /* B's events follow A's in the trace */
                if (h >= 2) {
                    LOAD(v, k + h + 1);
                    for (size_t j = 1; j < h; ++j) {       /* B has h-1 ranks: k+h+1 .. k+N-1 */
                        const int last = (j == h - 1);
                        if (!last) LOAD(x, k + h + 1 + j);
                        event = event_b++;
                        hop_receive(quant_rs, payload, v, block, last ? acc : x, w, codes, &scale);
                        RECORD(quant_rs);
                        memcpy(last ? acc : v, w, (size_t)block * sizeof(float));
                    }
                }
                /* chain A: k+h -> k+h-1 -> ... -> k+1 -> owner */
                LOAD(v, k + h);
                event = 0;
                for (size_t j = 1; j <= h; ++j) {
                    const int last = (j == h);
                    if (!last) LOAD(x, k + h - j);
                    hop_receive(quant_rs, payload, v, block, last ? acc : x, w, codes, &scale);
                    RECORD(quant_rs);
                    memcpy(last ? acc : v, w, (size_t)block * sizeof(float));
                }
            }
            /* acc is the owner's reduced block: fp32 if the hops were quantized, else a bf16 value */
            event = N - 1;
            if (quant_ag) {
                quantize_one_block_payload(acc, block, payload, codes, &scale);
                RECORD(1);
                for (int i = 0; i < block; ++i) {
                    uint16_t h16 = f32_to_bf16_rne(code_value(codes[i], payload) * scale);
                    for (size_t r = 0; r < N; ++r) out[r][base + (size_t)i] = h16;
                }
            } else {
                for (int i = 0; i < block; ++i) {
                    uint16_t h16 = f32_to_bf16_rne(acc[i]);
                    for (size_t r = 0; r < N; ++r) out[r][base + (size_t)i] = h16;
                }
            }
#undef LOAD
#undef RECORD
        }
    }
    free(v);
    free(codes);
    return ORACLE_OK;
}

/*
 * A-posteriori error bound of the quantized AllReduce against the exact sum,
 * from the scales of the trace: every quantize event j of a block moves a
 * value by at most half a quantization step scale_j (plus the fp32 rounding
 * of the multiply, the two divisions and the following fused add, together
 * below scale_j * 2^-14); a flushed block (scale 0) drops less than 2^-118
 * per element; the last bf16 rounding is 2^-9 relative, written against the
 * output as 2^-7.9; 2^-133 covers subnormal roundings.
 *
 *   bound[e] = sum_j c_j + 2^-7.9 * |out[e]| + 2^-133,
 *   c_j = scale_j * (0.5 + 2^-14) if scale_j > 0 else 2^-117.
 *
 * trace_scales as written by equarx_oracle_allreduce; out is any rank's output.
 */
int equarx_oracle_error_bound(const float *trace_scales, const uint16_t *out,
                              int nranks, size_t count, int block, double *bound)
{
    if (!trace_scales || !out || !bound) return ORACLE_ERR_NULL;
    int st = check_sim_args(nranks, count, block);
    if (st) return st;
    const size_t N = (size_t)nranks;
    const size_t shard = count / N;
    const size_t bps = shard / (size_t)block;
    const double rel_out = pow(2.0, -7.9);
    for (size_t k = 0; k < N; ++k) {
        for (size_t b = 0; b < bps; ++b) {
            double acc = 0.0;
            for (size_t j = 0; j < N; ++j) {
                double sc = (double)trace_scales[(k * N + j) * bps + b];
                acc += sc > 0.0 ? sc * (0.5 + 0x1p-14) : 0x1p-117;
            }
            for (int i = 0; i < block; ++i) {
                size_t e = k * shard + b * (size_t)block + (size_t)i;
                bound[e] = acc + rel_out * fabs((double)bf16_to_f32(out[e])) + 0x1p-133;
            }
        }
    }
    return ORACLE_OK;
}
