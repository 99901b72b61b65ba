/*
 * A plain C program that uses the library through include/equarx.h alone (no Python, no
 * torch): device memory from the CUDA runtime, the whole simulated AllReduce and the three
 * per-step entry points, compared word for word with the C oracle (linked by the test).
 * Exit code 0 = all comparisons equal.
 */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "equarx.h"

int equarx_oracle_allreduce(const uint16_t *const *in, uint16_t *const *out, int nranks, size_t count, int block,
                            float *trace_scales, int8_t *trace_codes, double *exact_sum);
int equarx_oracle_quantize_blocks(const uint16_t *x, size_t count, int block, int8_t *codes, float *scales);
int equarx_oracle_rs_step(const int8_t *codes_in, const float *scales_in, const uint16_t *local, size_t count,
                          int block, int8_t *codes_out, float *scales_out);
int equarx_oracle_ag_dequant(const int8_t *codes, const float *scales, size_t count, int block, uint16_t *out);

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { \
    fprintf(stderr, "CUDA error %d at %s:%d\n", (int)e_, __FILE__, __LINE__); return 2; } } while (0)
#define CHECK_EQ(x) do { int s_ = (x); if (s_ != EQUARX_OK) { \
    fprintf(stderr, "%s at %s:%d\n", equarx_status_string(s_), __FILE__, __LINE__); return 3; } } while (0)

/* bf16 words with a spread of exponents, finite, from a small linear congruential generator */
static uint16_t next_bf16(uint32_t *state)
{
    *state = *state * 1664525u + 1013904223u;
    uint32_t sign = (*state >> 31) << 15, mant = (*state >> 8) & 0x7Fu, exp = 120u + ((*state >> 16) % 12u);
    return (uint16_t)(sign | (exp << 7) | mant);
}

int main(void)
{
    enum { N = 4, BLOCK = 128, BPS = 9 };
    const size_t shard = (size_t)BLOCK * BPS, count = shard * N;
    uint32_t rng = 2024u;
    uint16_t *h_in[N], *h_out[N], *h_ref[N];
    void *d_in[N], *d_out[N];
    for (int r = 0; r < N; ++r) {
        h_in[r] = malloc(count * 2); h_out[r] = malloc(count * 2); h_ref[r] = malloc(count * 2);
        for (size_t i = 0; i < count; ++i) h_in[r][i] = next_bf16(&rng);
        CHECK_CUDA(cudaMalloc(&d_in[r], count * 2));
        CHECK_CUDA(cudaMalloc(&d_out[r], count * 2));
        CHECK_CUDA(cudaMemcpy(d_in[r], h_in[r], count * 2, cudaMemcpyHostToDevice));
    }
    /* the whole AllReduce, launch-per-step and pipelined */
    CHECK_EQ(equarx_oracle_allreduce((const uint16_t *const *)h_in, h_ref, N, count, BLOCK, NULL, NULL, NULL));
    for (int pipelined = 0; pipelined < 2; ++pipelined) {
        size_t wb = pipelined ? equarx_allreduce_sim_pipelined_workspace_bytes(N, count, BLOCK, 0)
                              : equarx_allreduce_sim_workspace_bytes(N, count, BLOCK, 0);
        void *ws;
        CHECK_CUDA(cudaMalloc(&ws, wb));
        if (pipelined)
            CHECK_EQ(equarx_allreduce_sim_pipelined((const void *const *)d_in, d_out, N, count, BLOCK, ws, wb, 0, NULL));
        else
            CHECK_EQ(equarx_allreduce_sim((const void *const *)d_in, d_out, N, count, BLOCK, ws, wb, 0, NULL));
        CHECK_CUDA(cudaDeviceSynchronize());
        for (int r = 0; r < N; ++r) {
            CHECK_CUDA(cudaMemcpy(h_out[r], d_out[r], count * 2, cudaMemcpyDeviceToHost));
            if (memcmp(h_out[r], h_ref[r], count * 2) != 0) {
                fprintf(stderr, "AllReduce output of rank %d differs (pipelined=%d)\n", r, pipelined);
                return 1;
            }
        }
        CHECK_CUDA(cudaFree(ws));
    }
    /* the per-step entry points: quantize rank 0's tensor, one hop with rank 1's, dequantize */
    {
        const size_t nb = count / BLOCK;
        int8_t *d_c0, *d_c1, *h_c = malloc(count), *r_c0 = malloc(count), *r_c1 = malloc(count);
        float *d_s0, *d_s1, *h_s = malloc(nb * 4), *r_s0 = malloc(nb * 4), *r_s1 = malloc(nb * 4);
        CHECK_CUDA(cudaMalloc((void **)&d_c0, count)); CHECK_CUDA(cudaMalloc((void **)&d_c1, count));
        CHECK_CUDA(cudaMalloc((void **)&d_s0, nb * 4)); CHECK_CUDA(cudaMalloc((void **)&d_s1, nb * 4));
        CHECK_EQ(equarx_quantize_blocks(d_in[0], count, BLOCK, d_c0, d_s0, NULL));
        CHECK_EQ(equarx_rs_step_dequant_add_requant(d_c0, d_s0, d_in[1], count, BLOCK, d_c1, d_s1, NULL));
        CHECK_EQ(equarx_ag_dequant(d_c1, d_s1, count, BLOCK, d_out[0], NULL));
        CHECK_CUDA(cudaDeviceSynchronize());
        CHECK_EQ(equarx_oracle_quantize_blocks(h_in[0], count, BLOCK, r_c0, r_s0));
        CHECK_EQ(equarx_oracle_rs_step(r_c0, r_s0, h_in[1], count, BLOCK, r_c1, r_s1));
        CHECK_EQ(equarx_oracle_ag_dequant(r_c1, r_s1, count, BLOCK, h_ref[0]));
        CHECK_CUDA(cudaMemcpy(h_c, d_c1, count, cudaMemcpyDeviceToHost));
        CHECK_CUDA(cudaMemcpy(h_s, d_s1, nb * 4, cudaMemcpyDeviceToHost));
        CHECK_CUDA(cudaMemcpy(h_out[0], d_out[0], count * 2, cudaMemcpyDeviceToHost));
        if (memcmp(h_c, r_c1, count) || memcmp(h_s, r_s1, nb * 4) || memcmp(h_out[0], h_ref[0], count * 2)) {
            fprintf(stderr, "per-step entry points differ from the oracle\n");
            return 1;
        }
    }
    /* host buffers in, host buffers out: pageable memory here, so the copies are synchronous */
    {
        void *stage;
        const size_t sb = equarx_allreduce_sim_host_staging_bytes(N, count);
        if (sb != 2 * count * N) return 1;
        CHECK_CUDA(cudaMalloc(&stage, sb));
        CHECK_EQ(equarx_oracle_allreduce((const uint16_t *const *)h_in, h_ref, N, count, BLOCK, NULL, NULL, NULL));
        for (int r = 0; r < N; ++r) memset(h_out[r], 0xEE, count * 2);
        CHECK_EQ(equarx_allreduce_sim_host((const void *const *)h_in, (void *const *)h_out, N, count, BLOCK, stage, sb,
                                           NULL));
        CHECK_CUDA(cudaDeviceSynchronize());
        for (int r = 0; r < N; ++r)
            if (memcmp(h_out[r], h_ref[r], count * 2) != 0) {
                fprintf(stderr, "host-buffer AllReduce output of rank %d differs\n", r);
                return 1;
            }
        if (equarx_allreduce_sim_host((const void *const *)h_in, (void *const *)h_out, N, count, BLOCK, stage, sb - 1,
                                      NULL) != EQUARX_ERR_WORKSPACE)
            return 1;
        CHECK_CUDA(cudaFree(stage));
    }
    /* the unordered single launch and the ring with one rank per device (all ranks hosted by this process) */
    {
        CHECK_EQ(equarx_oracle_allreduce((const uint16_t *const *)h_in, h_ref, N, count, BLOCK, NULL, NULL, NULL));
        for (int r = 0; r < N; ++r) CHECK_CUDA(cudaMemset(d_out[r], 0, count * 2));
        CHECK_EQ(equarx_allreduce_sim_pipelined_unordered((const void *const *)d_in, d_out, N, count, BLOCK, NULL));
        CHECK_CUDA(cudaDeviceSynchronize());
        for (int r = 0; r < N; ++r) {
            CHECK_CUDA(cudaMemcpy(h_out[r], d_out[r], count * 2, cudaMemcpyDeviceToHost));
            if (memcmp(h_out[r], h_ref[r], count * 2) != 0) { fprintf(stderr, "unordered launch: rank %d differs\n", r); return 1; }
        }
        void *boxes[N];
        uint32_t *status, h_status[4];
        const size_t box_bytes = equarx_ring_mailbox_bytes(N, count, BLOCK);
        if (box_bytes == 0) return 1;
        for (int r = 0; r < N; ++r) {
            CHECK_CUDA(cudaMalloc(&boxes[r], box_bytes));
            CHECK_CUDA(cudaMemset(boxes[r], 0, box_bytes));
            CHECK_CUDA(cudaMemset(d_out[r], 0, count * 2));
        }
        CHECK_CUDA(cudaMalloc((void **)&status, 16));
        CHECK_CUDA(cudaMemset(status, 0, 16));
        for (uint32_t epoch = 1; epoch <= 2; ++epoch)
            CHECK_EQ(equarx_ring_allreduce((const void *const *)d_in, d_out, 0, N, N, count, BLOCK, boxes, epoch, 0, status,
                                           NULL));
        CHECK_CUDA(cudaDeviceSynchronize());
        CHECK_CUDA(cudaMemcpy(h_status, status, 16, cudaMemcpyDeviceToHost));
        if (h_status[0] != 0) { fprintf(stderr, "ring: status %u\n", h_status[0]); return 1; }
        for (int r = 0; r < N; ++r) {
            CHECK_CUDA(cudaMemcpy(h_out[r], d_out[r], count * 2, cudaMemcpyDeviceToHost));
            if (memcmp(h_out[r], h_ref[r], count * 2) != 0) { fprintf(stderr, "ring: rank %d differs\n", r); return 1; }
            CHECK_CUDA(cudaFree(boxes[r]));
        }
        if (equarx_ring_allreduce((const void *const *)d_in, d_out, 0, N, N, count, BLOCK, boxes, 0, 0, status, NULL)
            != EQUARX_ERR_COUNT)           /* epoch 0 is refused */
            return 1;
        CHECK_CUDA(cudaFree(status));
    }
    /* an error path: a count that is not a multiple of nranks * block is refused before any launch */
    if (equarx_allreduce_sim((const void *const *)d_in, d_out, N, count + BLOCK, BLOCK, d_out[0], 1 << 20, 0, NULL)
        != EQUARX_ERR_COUNT)
        return 1;
    printf("c abi ok: N=%d count=%zu block=%d\n", (int)N, count, (int)BLOCK);
    return 0;
}
