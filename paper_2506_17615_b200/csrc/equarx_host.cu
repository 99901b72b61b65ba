// C ABI of the EQuARX hot-path library: argument validation, the ring step
// loop (full-loop reduce-scatter + quantized all-gather, Sections 3, 3.3, 3.4
// of arXiv 2506.17615) and the launches.  Declarations and the contract of
// every entry point are in include/equarx.h.
#include "equarx_kernels.cuh"

#include <algorithm>
#include <atomic>
#include <mutex>
#include <vector>
#include <cstdlib>
#include <cstring>

#include "../../include/equarx.h"

namespace {

using namespace equarx;

thread_local int g_last_cuda_error = 0;

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

inline bool overlap(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

inline int lanes_per_block(int block) {
    switch (block) {
        case 64: return 4;
        case 128: return 8;
        case 256: return 16;
        case 512: return 32;
        default: return 0;
    }
}

constexpr size_t kMaxCount = size_t(1) << 40;

inline int check_step_shape(size_t count, int block) {
    if (!lanes_per_block(block)) return EQUARX_ERR_BLOCK;
    if (count == 0 || count > kMaxCount || count % size_t(block) != 0) return EQUARX_ERR_COUNT;
    return EQUARX_OK;
}

inline int check_sim_shape(int nranks, size_t count, int block) {
    if (nranks < 1 || nranks > EQUARX_MAX_RANKS) return EQUARX_ERR_NRANKS;
    if (!lanes_per_block(block)) return EQUARX_ERR_BLOCK;
    if (count == 0 || count > kMaxCount || count % (size_t(nranks) * size_t(block)) != 0)
        return EQUARX_ERR_COUNT;
    return EQUARX_OK;
}

// Programmatic dependent launch is on unless EQUARX_PDL=0 (read once).
bool use_pdl() {
    static const bool on = [] {
        const char* e = std::getenv("EQUARX_PDL");
        return !(e && e[0] == '0');
    }();
    return on;
}

// Host-side fault injection for tests: with EQUARX_INJECT_LAUNCH_ERROR=<cudaError_t value> in the
// environment every launch is skipped and reports that error instead, so that the error path
// (status, equarx_last_cuda_error) can be exercised without making a GPU fault.
inline cudaError_t injected_launch_error() {
    const char* e = std::getenv("EQUARX_INJECT_LAUNCH_ERROR");
    return e ? cudaError_t(std::atoi(e)) : cudaSuccess;
}

template <typename Kernel, typename Args>
int launch(Kernel kernel, dim3 grid, const Args& args, cudaStream_t stream, bool dependent) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (dependent && use_pdl()) ? 1 : 0;
    cudaError_t e = injected_launch_error();
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, kernel, args);
    if (e != cudaSuccess) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    return EQUARX_OK;
}

inline dim3 grid_for(uint64_t shard, unsigned y) {
    const uint64_t groups = shard / kLaneElems;
    return dim3(unsigned((groups + kThreads - 1) / kThreads), y, 1);
}

template <bool FIRST, bool RECORDS>
int launch_step(int block, const StepArgs& a, unsigned nranks, cudaStream_t stream, bool dependent) {
    const dim3 grid = grid_for(a.shard, nranks);
    switch (block) {
        case 64: return launch(rs_step_kernel<4, FIRST, RECORDS>, grid, a, stream, dependent);
        case 128: return launch(rs_step_kernel<8, FIRST, RECORDS>, grid, a, stream, dependent);
        case 256: return launch(rs_step_kernel<16, FIRST, RECORDS>, grid, a, stream, dependent);
        default: return launch(rs_step_kernel<32, FIRST, RECORDS>, grid, a, stream, dependent);
    }
}

template <bool RECORDS>
int launch_gather(int block, const GatherArgs& a, cudaStream_t stream, bool dependent) {
    const dim3 grid = grid_for(a.shard, a.nranks);
    switch (block) {
        case 64: return launch(ag_dequant_kernel<4, RECORDS>, grid, a, stream, dependent);
        case 128: return launch(ag_dequant_kernel<8, RECORDS>, grid, a, stream, dependent);
        case 256: return launch(ag_dequant_kernel<16, RECORDS>, grid, a, stream, dependent);
        default: return launch(ag_dequant_kernel<32, RECORDS>, grid, a, stream, dependent);
    }
}

// Launch geometry of a persistent kernel depends on the device (SM count) and on the kernel's
// occupancy; both are constant for the life of the process, so they are looked up once per
// (device, kernel) and remembered: the queries cost about as much as the launch itself.
struct Residency {
    int sms = 0, occ = 0, coop = 0;
};

cudaError_t residency_of(const void* kernel, int threads, Residency& out) {
    struct Entry {
        int dev;
        const void* kernel;
        Residency r;
    };
    static std::mutex mu;
    static std::vector<Entry> seen;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    {
        std::lock_guard<std::mutex> lock(mu);
        for (const Entry& en : seen)
            if (en.dev == dev && en.kernel == kernel) {
                out = en.r;
                return cudaSuccess;
            }
    }
    Residency r;
    e = cudaDeviceGetAttribute(&r.sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&r.coop, cudaDevAttrCooperativeLaunch, dev);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r.occ, kernel, threads, 0);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    seen.push_back(Entry{dev, kernel, r});
    out = r;
    return cudaSuccess;
}

// Persistent grid of the single-launch kernels: a whole number of CTAs per SM (measured: a grid that
// balances the warps' tile counts but loads the SMs unevenly is 2 % slower at 88 MB per rank and no
// faster at 16 MB), the count per SM that needs the fewest rounds of tiles and, among those, the
// smallest; never more CTAs than there are tiles to carry.
inline uint64_t persistent_grid(uint64_t tiles, uint64_t warps_per_cta, int sms, int occ) {
    uint64_t best = 0, best_rounds = ~uint64_t(0);
    for (int c = 1; c <= occ; ++c) {
        const uint64_t ctas = uint64_t(sms) * c, w = ctas * warps_per_cta;
        const uint64_t rounds = (tiles + w - 1) / w;
        if (rounds < best_rounds) {
            best_rounds = rounds;
            best = ctas;
        }
    }
    return std::min<uint64_t>(best, (tiles + warps_per_cta - 1) / warps_per_cta);
}

// bytes of one message slot in the record layout: one 544-byte record per 512-element tile
inline size_t slot_bytes(size_t shard) { return (shard + kTileElems - 1) / kTileElems * size_t(kRecordBytes); }

// in/out tables of a simulation: NULLs, alignment, overlap.  out[r] == in[r] is the
// one overlap allowed.
int check_tables(const void* const* in, void* const* out, int nranks, size_t bytes,
                 const void* ws, size_t ws_bytes) {
    if (!in || !out) return EQUARX_ERR_NULL;
    for (int r = 0; r < nranks; ++r)
        if (!in[r] || !out[r]) return EQUARX_ERR_NULL;
    for (int r = 0; r < nranks; ++r)
        if (!aligned(in[r], 32) || !aligned(out[r], 32)) return EQUARX_ERR_ALIGN;
    for (int r = 0; r < nranks; ++r) {
        for (int q = 0; q < nranks; ++q) {
            if (q != r && overlap(out[r], bytes, out[q], bytes)) return EQUARX_ERR_ALIAS;
            if (overlap(out[r], bytes, in[q], bytes) && !(q == r && out[r] == in[r]))
                return EQUARX_ERR_ALIAS;
        }
        if (ws && (overlap(ws, ws_bytes, in[r], bytes) || overlap(ws, ws_bytes, out[r], bytes)))
            return EQUARX_ERR_ALIAS;
    }
    return EQUARX_OK;
}

template <int LPB, int PAYLOAD>
const void* flavour_kernel_for(int flavour) {
    switch (flavour & 7) {
        case 2: return reinterpret_cast<const void*>(flavour_kernel<LPB, false, true, false, PAYLOAD>);
        case 3: return reinterpret_cast<const void*>(flavour_kernel<LPB, true, true, false, PAYLOAD>);
        case 4: return reinterpret_cast<const void*>(flavour_kernel<LPB, false, false, true, PAYLOAD>);
        case 5: return reinterpret_cast<const void*>(flavour_kernel<LPB, true, false, true, PAYLOAD>);
        case 6: return reinterpret_cast<const void*>(flavour_kernel<LPB, false, true, true, PAYLOAD>);
        case 7: return reinterpret_cast<const void*>(flavour_kernel<LPB, true, true, true, PAYLOAD>);
        // nothing is quantized: the payload type does not matter
        case 1: return reinterpret_cast<const void*>(flavour_kernel<LPB, true, false, false, 1>);
        default: return reinterpret_cast<const void*>(flavour_kernel<LPB, false, false, false, 1>);
    }
}

template <int LPB>
const void* flavour_kernel_for(int flavour) {
    if (flavour & EQUARX_FLAVOUR_E4M3) return flavour_kernel_for<LPB, 2>(flavour);
    if (flavour & EQUARX_FLAVOUR_E5M2) return flavour_kernel_for<LPB, 3>(flavour);
    return flavour_kernel_for<LPB, 1>(flavour);
}

// the same flavours with the messages kept in registers (no trace)
template <int LPB, int PAYLOAD>
const void* flavour_fused_kernel_for(int flavour) {
    switch (flavour & 7) {
        case 2: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, false, true, false, PAYLOAD>);
        case 3: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, true, true, false, PAYLOAD>);
        case 4: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, false, false, true, PAYLOAD>);
        case 5: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, true, false, true, PAYLOAD>);
        case 6: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, false, true, true, PAYLOAD>);
        case 7: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, true, true, true, PAYLOAD>);
        case 1: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, true, false, false, 1>);
        default: return reinterpret_cast<const void*>(flavour_fused_kernel<LPB, false, false, false, 1>);
    }
}

template <int LPB>
const void* flavour_fused_kernel_for(int flavour) {
    if (flavour & EQUARX_FLAVOUR_E4M3) return flavour_fused_kernel_for<LPB, 2>(flavour);
    if (flavour & EQUARX_FLAVOUR_E5M2) return flavour_fused_kernel_for<LPB, 3>(flavour);
    return flavour_fused_kernel_for<LPB, 1>(flavour);
}

// a valid flavour: any of the three schedule bits, at most one payload bit, and a payload bit
// only together with a quantized stage
inline bool flavour_ok(int flavour) {
    if (flavour < 0 || flavour > 31) return false;
    const bool e4 = flavour & EQUARX_FLAVOUR_E4M3, e5 = flavour & EQUARX_FLAVOUR_E5M2;
    if (e4 && e5) return false;
    if ((e4 || e5) && !(flavour & (EQUARX_FLAVOUR_QUANT_RS | EQUARX_FLAVOUR_QUANT_AG))) return false;
    return true;
}

}  // namespace

extern "C" {

const char* equarx_status_string(int status) {
    switch (status) {
        case EQUARX_OK: return "EQUARX_OK";
        case EQUARX_ERR_NULL: return "EQUARX_ERR_NULL: a required pointer is NULL";
        case EQUARX_ERR_NRANKS: return "EQUARX_ERR_NRANKS: nranks outside [1, 64]";
        case EQUARX_ERR_BLOCK: return "EQUARX_ERR_BLOCK: block must be 64, 128, 256 or 512";
        case EQUARX_ERR_COUNT: return "EQUARX_ERR_COUNT: count is 0, too large or not a multiple of the required unit";
        case EQUARX_ERR_ALIGN: return "EQUARX_ERR_ALIGN: a pointer is not aligned as required";
        case EQUARX_ERR_WORKSPACE: return "EQUARX_ERR_WORKSPACE: workspace too small";
        case EQUARX_ERR_ALIAS: return "EQUARX_ERR_ALIAS: buffers overlap";
        case EQUARX_ERR_CUDA: return "EQUARX_ERR_CUDA: a kernel launch failed";
        case EQUARX_ERR_FLAVOUR: return "EQUARX_ERR_FLAVOUR: flavour must be a combination of the EQUARX_FLAVOUR_* bits";
        case EQUARX_ERR_STATIC_LIMIT:
            return "EQUARX_ERR_STATIC_LIMIT: problem needs more than the 16 MiB built-in workspace";
        default: return "EQUARX: unknown status";
    }
}

int equarx_last_cuda_error(void) { return g_last_cuda_error; }

int equarx_quantize_blocks(const void* x_bf16, size_t count, int block, int8_t* codes, float* scales,
                           equarx_stream_t stream) {
    if (!x_bf16 || !codes || !scales) return EQUARX_ERR_NULL;
    if (int st = check_step_shape(count, block)) return st;
    if (!aligned(x_bf16, 32) || !aligned(codes, 16) || !aligned(scales, 4)) return EQUARX_ERR_ALIGN;
    if (overlap(x_bf16, 2 * count, codes, count) || overlap(x_bf16, 2 * count, scales, 4 * (count / block)) ||
        overlap(codes, count, scales, 4 * (count / block)))
        return EQUARX_ERR_ALIAS;
    StepArgs a = {};
    a.neg_zero = -0.0f;
    a.x[0] = x_bf16;
    a.codes_out = codes;
    a.scales_out = scales;
    a.shard = count;
    a.bps = count / size_t(block);
    return launch_step<true, false>(block, a, 1, stream, false);
}

int equarx_rs_step_dequant_add_requant(const int8_t* codes_in, const float* scales_in, const void* local_bf16,
                                       size_t count, int block, int8_t* codes_out, float* scales_out,
                                       equarx_stream_t stream) {
    if (!codes_in || !scales_in || !local_bf16 || !codes_out || !scales_out) return EQUARX_ERR_NULL;
    if (int st = check_step_shape(count, block)) return st;
    if (!aligned(local_bf16, 32) || !aligned(codes_in, 16) || !aligned(codes_out, 16) || !aligned(scales_in, 4) ||
        !aligned(scales_out, 4))
        return EQUARX_ERR_ALIGN;
    const size_t sb = 4 * (count / size_t(block));
    const void* bufs[5] = {codes_in, scales_in, local_bf16, codes_out, scales_out};
    const size_t lens[5] = {count, sb, 2 * count, count, sb};
    for (int i = 0; i < 5; ++i)
        for (int j = 3; j < 5; ++j)
            if (i != j && overlap(bufs[i], lens[i], bufs[j], lens[j])) return EQUARX_ERR_ALIAS;
    StepArgs a = {};
    a.neg_zero = -0.0f;
    a.x[0] = local_bf16;
    a.codes_in = codes_in;
    a.scales_in = scales_in;
    a.codes_out = codes_out;
    a.scales_out = scales_out;
    a.shard = count;
    a.bps = count / size_t(block);
    return launch_step<false, false>(block, a, 1, stream, false);
}

int equarx_ag_dequant(const int8_t* codes, const float* scales, size_t count, int block, void* out_bf16,
                      equarx_stream_t stream) {
    if (!codes || !scales || !out_bf16) return EQUARX_ERR_NULL;
    if (int st = check_step_shape(count, block)) return st;
    if (!aligned(out_bf16, 32) || !aligned(codes, 16) || !aligned(scales, 4)) return EQUARX_ERR_ALIGN;
    if (overlap(out_bf16, 2 * count, codes, count) || overlap(out_bf16, 2 * count, scales, 4 * (count / block)))
        return EQUARX_ERR_ALIAS;
    GatherArgs a = {};
    a.out[0] = out_bf16;
    a.codes = codes;
    a.scales = scales;
    a.shard = count;
    a.bps = count / size_t(block);
    a.nranks = 1;
    return launch_gather<false>(block, a, stream, false);
}

size_t equarx_allreduce_sim_workspace_bytes(int nranks, size_t count, int block, int keep_trace) {
    if (check_sim_shape(nranks, count, block) != EQUARX_OK) return 0;
    const size_t N = size_t(nranks);
    const size_t slots = keep_trace ? N * N : 2 * N;
    return slots * slot_bytes(count / N);
}

int equarx_allreduce_sim(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count, int block,
                         void* workspace, size_t workspace_bytes, int keep_trace, equarx_stream_t stream) {
    return equarx_allreduce_sim_range(in_bf16, out_bf16, nranks, count, block, workspace, workspace_bytes,
                                      keep_trace, 0, nranks, stream);
}

int equarx_allreduce_sim_range(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count,
                               int block, void* workspace, size_t workspace_bytes, int keep_trace,
                               int first_launch, int last_launch, equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (first_launch < 0 || first_launch > last_launch || last_launch > nranks) return EQUARX_ERR_COUNT;
    if (!workspace) return EQUARX_ERR_NULL;
    const size_t need = equarx_allreduce_sim_workspace_bytes(nranks, count, block, keep_trace);
    if (workspace_bytes < need) return EQUARX_ERR_WORKSPACE;
    if (!aligned(workspace, 32)) return EQUARX_ERR_ALIGN;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, workspace, need)) return st;

    const uint32_t N = uint32_t(nranks);
    const size_t shard = count / N;
    int8_t* records = static_cast<int8_t*>(workspace);

    // shard that rank r sends at step s, and where that message is kept
    auto shard_of = [N](uint32_t s, uint32_t r) { return (r + 2 * N - 1 - s % N) % N; };
    auto slot_of = [&](uint32_t s, uint32_t r) {
        return keep_trace ? shard_of(s, r) * N + s : shard_of(s, r) * 2 + (s & 1u);
    };

    StepArgs a = {};
    a.neg_zero = -0.0f;
    a.codes_in = records;
    a.codes_out = records;
    a.shard = shard;
    a.bps = slot_bytes(shard);
    const uint32_t first = uint32_t(first_launch), last = uint32_t(last_launch);
    for (uint32_t s = first; s < N && s <= last; ++s) {
        for (uint32_t r = 0; r < N; ++r) {
            a.x[r] = static_cast<const char*>(in_bf16[r]) + size_t(shard_of(s, r)) * shard * 2;
            a.out_slot[r] = slot_of(s, r);
            a.in_slot[r] = s ? slot_of(s - 1, (r + N - 1) % N) : 0;
        }
        // step 0 waits for the stream's earlier work before its first load, so it can always be a
        // programmatic dependent; a later step loads its shard ahead of the wait and may only overlap
        // a launch of this same call
        const int st = s == 0 ? launch_step<true, true>(block, a, N, stream, true)
                              : launch_step<false, true>(block, a, N, stream, s > first);
        if (st) return st;
    }
    if (last < N) return EQUARX_OK;

    GatherArgs g = {};
    for (uint32_t k = 0; k < N; ++k) {
        g.out[k] = out_bf16[k];
        g.slot[k] = slot_of(N - 1, k);     // after step N-1 rank k holds shard k
    }
    g.codes = records;
    g.shard = shard;
    g.bps = slot_bytes(shard);
    g.nranks = N;
    return launch_gather<true>(block, g, stream, first < N);
}

size_t equarx_allreduce_sim_pipelined_workspace_bytes(int nranks, size_t count, int block, int keep_trace) {
    if (check_sim_shape(nranks, count, block) != EQUARX_OK) return 0;
    if (keep_trace) return equarx_allreduce_sim_workspace_bytes(nranks, count, block, 1);
    return size_t(EQUARX_PIPELINE_MIN_WORKSPACE_BYTES);      // not touched: the chain-fused kernel needs no scratch
}

}  // extern "C"

namespace {
// the single-launch schedule on validated arguments (workspace: the trace, or unused)
int launch_pipelined(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count, int block,
                     void* workspace, int keep_trace, cudaStream_t stream, bool quantized = true,
                     bool unordered = false) {
    const uint32_t N = uint32_t(nranks);
    const size_t shard = count / N;
    PipeArgs a = {};
    a.neg_zero = -0.0f;
    for (uint32_t r = 0; r < N; ++r) {
        a.in[r] = in_bf16[r];
        a.out[r] = out_bf16[r];
    }
    a.records = static_cast<char*>(workspace);
    a.unordered = (unordered && !keep_trace) ? 1u : 0u;
    a.shard = shard;
    a.tiles_per_shard = (shard + kTileElems - 1) / kTileElems;
    a.nranks = N;

    constexpr int D = kFusedDepth;
    // register budget of the chain-fused kernel: see chain_fused_kernel
    const bool large = 2.0 * double(count) * double(nranks) > 200e6;
    const void* kernel = nullptr;
#define EQX_FUSED(L, Q) (large ? reinterpret_cast<const void*>(chain_fused_kernel<L, D, Q, 16>) \
                               : reinterpret_cast<const void*>(chain_fused_kernel<L, D, Q, 18>))
#define EQX_PICK(L) \
    kernel = keep_trace ? reinterpret_cast<const void*>(pipelined_kernel<L>) : quantized ? EQX_FUSED(L, true) : EQX_FUSED(L, false)
    switch (block) {
        case 64: EQX_PICK(4); break;
        case 128: EQX_PICK(8); break;
        case 256: EQX_PICK(16); break;
        default: EQX_PICK(32); break;
    }
#undef EQX_FUSED
#undef EQX_PICK
    // persistent grid: a whole number of CTAs per SM
    Residency res;
    cudaError_t e = residency_of(kernel, kPipeThreads, res);
    const int sms = res.sms, occ = res.occ;
    if (e != cudaSuccess || sms < 1 || occ < 1) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    const uint64_t best_ctas = persistent_grid(a.tiles_per_shard * N, kPipeThreads / 32, sms, occ);

    // programmatic dependent launch hides the launch latency behind the previous kernel's tail; the
    // kernel itself waits for that kernel to complete before its first memory access
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(best_ctas));
    cfg.blockDim = dim3(kPipeThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = use_pdl() ? 1 : 0;
    void* params[1] = {&a};
    e = injected_launch_error();
    if (e == cudaSuccess) e = cudaLaunchKernelExC(&cfg, kernel, params);
    if (e != cudaSuccess) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    return EQUARX_OK;
}
}  // namespace

extern "C" {

int equarx_allreduce_sim_pipelined(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count,
                                   int block, void* workspace, size_t workspace_bytes, int keep_trace,
                                   equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (!workspace) return EQUARX_ERR_NULL;
    const size_t need = equarx_allreduce_sim_pipelined_workspace_bytes(nranks, count, block, keep_trace);
    if (workspace_bytes < need) return EQUARX_ERR_WORKSPACE;
    if (!aligned(workspace, 32)) return EQUARX_ERR_ALIGN;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, workspace, need)) return st;
    return launch_pipelined(in_bf16, out_bf16, nranks, count, block, workspace, keep_trace, stream);
}

int equarx_allreduce_sim_pipelined_unordered(const void* const* in_bf16, void* const* out_bf16, int nranks,
                                             size_t count, int block, equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, nullptr, 0)) return st;
    return launch_pipelined(in_bf16, out_bf16, nranks, count, block, nullptr, 0, stream, true, true);
}

size_t equarx_allreduce_sim_host_staging_bytes(int nranks, size_t count) {
    if (nranks < 1 || nranks > EQUARX_MAX_RANKS || count == 0 || count > kMaxCount) return 0;
    return 2 * count * size_t(nranks);
}

int equarx_allreduce_sim_host(const void* const* host_in, void* const* host_out, int nranks, size_t count,
                              int block, void* staging, size_t staging_bytes, equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (!host_in || !host_out || !staging) return EQUARX_ERR_NULL;
    for (int r = 0; r < nranks; ++r)
        if (!host_in[r] || !host_out[r]) return EQUARX_ERR_NULL;
    const size_t bytes = 2 * count;
    if (staging_bytes < bytes * size_t(nranks)) return EQUARX_ERR_WORKSPACE;
    if (!aligned(staging, 32)) return EQUARX_ERR_ALIGN;
    for (int r = 0; r < nranks; ++r) {
        if (!aligned(host_in[r], 2) || !aligned(host_out[r], 2)) return EQUARX_ERR_ALIGN;
        for (int q = 0; q < nranks; ++q) {
            if (q != r && overlap(host_out[r], bytes, host_out[q], bytes)) return EQUARX_ERR_ALIAS;
            if (overlap(host_out[r], bytes, host_in[q], bytes) && !(q == r && host_out[r] == host_in[r]))
                return EQUARX_ERR_ALIAS;
        }
    }
    const void* dev_in[EQUARX_MAX_RANKS];
    void* dev_out[EQUARX_MAX_RANKS];
    for (int r = 0; r < nranks; ++r) dev_in[r] = dev_out[r] = static_cast<char*>(staging) + size_t(r) * bytes;

    auto failed = [](cudaError_t e) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    };
    cudaError_t e = injected_launch_error();
    if (e != cudaSuccess) return failed(e);
    for (int r = 0; r < nranks; ++r) {
        e = cudaMemcpyAsync(dev_out[r], host_in[r], bytes, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return failed(e);
    }
    // reduced in place in the staging buffer; the chain-fused kernel needs no workspace
    if (int st = launch_pipelined(dev_in, dev_out, nranks, count, block, nullptr, 0, stream)) return st;
    for (int r = 0; r < nranks; ++r) {
        e = cudaMemcpyAsync(host_out[r], dev_out[r], bytes, cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) return failed(e);
    }
    return EQUARX_OK;
}

size_t equarx_allreduce_sim_flavour_workspace_bytes(int nranks, size_t count, int block, int flavour,
                                                    int keep_trace) {
    if (check_sim_shape(nranks, count, block) != EQUARX_OK) return 0;
    if (!flavour_ok(flavour)) return 0;
    if ((flavour & EQUARX_FLAVOUR_SEMI_LOOP) && nranks % 2 != 0) return 0;
    if (!keep_trace) return size_t(EQUARX_PIPELINE_MIN_WORKSPACE_BYTES);   // messages stay in registers
    return size_t(EQUARX_FLAVOUR_FIFO_BYTES) + equarx_allreduce_sim_workspace_bytes(nranks, count, block, 1);
}

int equarx_allreduce_sim_flavour(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count,
                                 int block, int flavour, void* workspace, size_t workspace_bytes, int keep_trace,
                                 equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (!flavour_ok(flavour)) return EQUARX_ERR_FLAVOUR;
    if ((flavour & EQUARX_FLAVOUR_SEMI_LOOP) && nranks % 2 != 0) return EQUARX_ERR_NRANKS;
    if (!workspace) return EQUARX_ERR_NULL;
    const size_t need = equarx_allreduce_sim_flavour_workspace_bytes(nranks, count, block, flavour, keep_trace);
    if (workspace_bytes < need) return EQUARX_ERR_WORKSPACE;
    if (!aligned(workspace, 32)) return EQUARX_ERR_ALIGN;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, workspace, need)) return st;

    const uint32_t N = uint32_t(nranks);
    const size_t shard = count / N;
    if (!keep_trace) {
        // the full loop with both stages quantized (int8) and the unquantized full loop have the tuned kernel
        const int sched = flavour & 7;
        const bool fp8 = flavour & (EQUARX_FLAVOUR_E4M3 | EQUARX_FLAVOUR_E5M2);
        if (sched == 0 || (sched == (EQUARX_FLAVOUR_QUANT_RS | EQUARX_FLAVOUR_QUANT_AG) && !fp8))
            return launch_pipelined(in_bf16, out_bf16, nranks, count, block, nullptr, 0, stream, sched != 0);
    }
    FlavourArgs a = {};
    a.neg_zero = -0.0f;
    for (uint32_t r = 0; r < N; ++r) {
        a.in[r] = in_bf16[r];
        a.out[r] = out_bf16[r];
    }
    a.fifo = keep_trace ? static_cast<char*>(workspace) : nullptr;
    a.trace = keep_trace ? static_cast<char*>(workspace) + size_t(EQUARX_FLAVOUR_FIFO_BYTES) : nullptr;
    a.shard = shard;
    a.tiles_per_shard = (shard + kTileElems - 1) / kTileElems;
    a.nranks = N;

    const void* kernel = nullptr;
    switch (block) {
        case 64: kernel = keep_trace ? flavour_kernel_for<4>(flavour) : flavour_fused_kernel_for<4>(flavour); break;
        case 128: kernel = keep_trace ? flavour_kernel_for<8>(flavour) : flavour_fused_kernel_for<8>(flavour); break;
        case 256: kernel = keep_trace ? flavour_kernel_for<16>(flavour) : flavour_fused_kernel_for<16>(flavour); break;
        default: kernel = keep_trace ? flavour_kernel_for<32>(flavour) : flavour_fused_kernel_for<32>(flavour); break;
    }
    Residency res;
    cudaError_t e = residency_of(kernel, kPipeThreads, res);
    const int sms = res.sms, occ = res.occ;
    if (e != cudaSuccess || sms < 1 || occ < 1) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    const uint64_t wpc = kPipeThreads / 32;
    uint64_t ctas = persistent_grid(a.tiles_per_shard * N, wpc, sms, occ);
    if (keep_trace) ctas = std::min<uint64_t>(ctas, uint64_t(EQUARX_FLAVOUR_FIFO_BYTES) / (2 * kFifoEntryBytes) / wpc);
    if (keep_trace) {                                  // events that this flavour does not quantize stay zero
        e = cudaMemsetAsync(a.trace, 0, need - size_t(EQUARX_FLAVOUR_FIFO_BYTES), stream);
        if (e != cudaSuccess) {
            g_last_cuda_error = int(e);
            (void)cudaGetLastError();
            return EQUARX_ERR_CUDA;
        }
    }
    void* params[1] = {&a};
    e = injected_launch_error();
    if (e == cudaSuccess) e = cudaLaunchKernel(kernel, dim3(unsigned(ctas)), dim3(kPipeThreads), params, 0, stream);
    if (e != cudaSuccess) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    return EQUARX_OK;
}

size_t equarx_ring_mailbox_bytes(int nranks, size_t count, int block) {
    if (check_sim_shape(nranks, count, block) != EQUARX_OK) return 0;
    const size_t N = size_t(nranks);
    const size_t tiles = (count / N + kTileElems - 1) / kTileElems;
    const size_t slots = 2 * N - 1;
    const size_t bytes = slots * tiles * size_t(kRecordBytes) + slots * tiles * sizeof(uint32_t);
    return (bytes + 255) / 256 * 256;
}

int equarx_ring_allreduce(const void* const* in_bf16, void* const* out_bf16, int rank_first, int ranks_here,
                          int nranks, size_t count, int block, void* const* mailboxes, uint32_t epoch,
                          uint64_t timeout_ns, uint32_t* status, equarx_stream_t stream) {
    if (int st = check_sim_shape(nranks, count, block)) return st;
    if (rank_first < 0 || ranks_here < 1 || rank_first + ranks_here > nranks) return EQUARX_ERR_NRANKS;
    if (epoch == 0) return EQUARX_ERR_COUNT;
    if (!in_bf16 || !out_bf16 || !mailboxes || !status) return EQUARX_ERR_NULL;
    const size_t bytes = 2 * count, box_bytes = equarx_ring_mailbox_bytes(nranks, count, block);
    for (int i = 0; i < ranks_here; ++i)
        if (!in_bf16[i] || !out_bf16[i]) return EQUARX_ERR_NULL;
    for (int q = 0; q < nranks; ++q)
        if (!mailboxes[q]) return EQUARX_ERR_NULL;
    if (!aligned(status, 16)) return EQUARX_ERR_ALIGN;
    for (int i = 0; i < ranks_here; ++i)
        if (!aligned(in_bf16[i], 32) || !aligned(out_bf16[i], 32)) return EQUARX_ERR_ALIGN;
    for (int q = 0; q < nranks; ++q)
        if (!aligned(mailboxes[q], 32)) return EQUARX_ERR_ALIGN;
    for (int i = 0; i < ranks_here; ++i) {
        for (int j = 0; j < ranks_here; ++j) {
            if (j != i && overlap(out_bf16[i], bytes, out_bf16[j], bytes)) return EQUARX_ERR_ALIAS;
            if (overlap(out_bf16[i], bytes, in_bf16[j], bytes) && !(j == i && out_bf16[i] == in_bf16[j]))
                return EQUARX_ERR_ALIAS;
        }
        for (int q = 0; q < nranks; ++q)
            if (overlap(mailboxes[q], box_bytes, in_bf16[i], bytes) || overlap(mailboxes[q], box_bytes, out_bf16[i], bytes))
                return EQUARX_ERR_ALIAS;
    }
    for (int q = 0; q < nranks; ++q)
        for (int p = q + 1; p < nranks; ++p)
            if (overlap(mailboxes[q], box_bytes, mailboxes[p], box_bytes)) return EQUARX_ERR_ALIAS;

    const uint32_t N = uint32_t(nranks);
    RingArgs a = {};
    a.neg_zero = -0.0f;
    for (int i = 0; i < ranks_here; ++i) {
        a.in[i] = in_bf16[i];
        a.out[i] = out_bf16[i];
    }
    for (uint32_t q = 0; q < N; ++q) a.mailbox[q] = static_cast<char*>(mailboxes[q]);
    a.status = status;
    a.shard = count / N;
    a.tiles_per_shard = (a.shard + kTileElems - 1) / kTileElems;
    a.timeout_ns = timeout_ns ? timeout_ns : 1000000000ull;
    a.nranks = N;
    a.rank_first = uint32_t(rank_first);
    a.ranks_here = uint32_t(ranks_here);
    a.epoch = epoch;

    const void* kernel = nullptr;
    switch (block) {
        case 64: kernel = reinterpret_cast<const void*>(ring_rank_kernel<4>); break;
        case 128: kernel = reinterpret_cast<const void*>(ring_rank_kernel<8>); break;
        case 256: kernel = reinterpret_cast<const void*>(ring_rank_kernel<16>); break;
        default: kernel = reinterpret_cast<const void*>(ring_rank_kernel<32>); break;
    }
    auto failed = [](cudaError_t e) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    };
    Residency res;
    cudaError_t e = residency_of(kernel, kRingThreads, res);
    const int sms = res.sms, occ = res.occ, coop = res.coop;
    if (e != cudaSuccess) return failed(e);
    if (sms < 1 || occ < 1 || !coop) return failed(cudaErrorCooperativeLaunchTooLarge);
    // every hosted rank gets the same number of CTAs and all of them must be resident at once
    const uint64_t resident = uint64_t(sms) * uint64_t(occ);
    const uint64_t wpc = kRingThreads / 32;
    uint64_t per_rank = resident / uint64_t(ranks_here);
    per_rank = std::min<uint64_t>(per_rank, (a.tiles_per_shard + wpc - 1) / wpc);
    if (per_rank < 1) return failed(cudaErrorCooperativeLaunchTooLarge);
    a.ctas_per_rank = uint32_t(per_rank);
    void* params[1] = {&a};
    e = injected_launch_error();
    if (e == cudaSuccess)
        e = cudaLaunchCooperativeKernel(kernel, dim3(unsigned(per_rank * uint64_t(ranks_here))), dim3(kRingThreads),
                                        params, 0, stream);
    if (e != cudaSuccess) return failed(e);
    return EQUARX_OK;
}

size_t equarx_allreduce_sim_bf16_workspace_bytes(int nranks, size_t count) {
    if (nranks < 1 || nranks > EQUARX_MAX_RANKS) return 0;
    if (count == 0 || count > kMaxCount || count % (size_t(nranks) * kLaneElems) != 0) return 0;
    return 4 * count;
}

int equarx_allreduce_sim_bf16(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count,
                              void* workspace, size_t workspace_bytes, equarx_stream_t stream) {
    if (nranks < 1 || nranks > EQUARX_MAX_RANKS) return EQUARX_ERR_NRANKS;
    if (count == 0 || count > kMaxCount || count % (size_t(nranks) * kLaneElems) != 0) return EQUARX_ERR_COUNT;
    if (!workspace) return EQUARX_ERR_NULL;
    const size_t need = 4 * count;
    if (workspace_bytes < need) return EQUARX_ERR_WORKSPACE;
    if (!aligned(workspace, 32)) return EQUARX_ERR_ALIGN;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, workspace, need)) return st;

    const uint32_t N = uint32_t(nranks);
    const size_t shard = count / N;
    char* ws = static_cast<char*>(workspace);
    auto shard_of = [N](uint32_t s, uint32_t r) { return (r + 2 * N - 1 - s % N) % N; };
    auto msg = [&](uint32_t s, uint32_t r) { return ws + (size_t(s & 1u) * N + r) * shard * 2; };

    Bf16StepArgs a = {};
    a.shard = shard;
    for (uint32_t s = 1; s < N; ++s) {
        for (uint32_t r = 0; r < N; ++r) {
            const uint32_t left = (r + N - 1) % N, k = shard_of(s, r);
            a.local[r] = static_cast<const char*>(in_bf16[r]) + size_t(k) * shard * 2;
            // step 0 sends the raw shard: the first hop reads the neighbour's input in place
            a.recv[r] = s == 1 ? static_cast<const char*>(in_bf16[left]) + size_t(k) * shard * 2 : msg(s - 1, left);
            a.send[r] = msg(s, r);
        }
        if (int st = launch(bf16_step_kernel, grid_for(shard, N), a, stream, s > 1)) return st;
    }
    Bf16GatherArgs g = {};
    g.shard = shard;
    g.nranks = N;
    for (uint32_t k = 0; k < N; ++k) {
        g.out[k] = out_bf16[k];
        g.src[k] = N == 1 ? in_bf16[0] : msg(N - 1, k);
    }
    return launch(bf16_gather_kernel, grid_for(shard, N), g, stream, N > 1);
}

// ---------------------------------------------------------------------------------
// Workspace-free variant for callers that cannot provide (or allocate) scratch memory.
// The hop messages go to a fixed array that is part of this library's device image,
// so every GPU that loads the library holds these 16 MiB until the process exits.
//
// `g_static_workspace` below is only a host-side handle when it is named in host
// code: it is NOT a device address and must never be passed to a kernel as is.  The
// device address is looked up once per device with cudaGetSymbolAddress while that
// device is current, and it is that address which goes into the kernel arguments.
static __device__ __align__(256) unsigned char g_static_workspace[EQUARX_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// device address of g_static_workspace, per device ordinal (every thread that sets it stores the same value)
std::atomic<void*> g_static_ptr[kMaxDevices];
}  // namespace

int equarx_allreduce_sim_static(const void* const* in_bf16, void* const* out_bf16, int nranks, size_t count,
                                int block, equarx_stream_t stream) {
    // host-side validation first: no CUDA call is made for arguments that are rejected
    if (int st = check_sim_shape(nranks, count, block)) return st;
    const size_t need = equarx_allreduce_sim_workspace_bytes(nranks, count, block, 0);
    if (need > size_t(EQUARX_STATIC_WORKSPACE_BYTES)) return EQUARX_ERR_STATIC_LIMIT;
    if (int st = check_tables(in_bf16, out_bf16, nranks, 2 * count, nullptr, 0)) return st;

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess && (dev < 0 || dev >= kMaxDevices)) e = cudaErrorInvalidDevice;
    void* ws = nullptr;
    if (e == cudaSuccess) {
        ws = g_static_ptr[dev].load(std::memory_order_relaxed);
        if (ws == nullptr) {
            // set-up, once per device, with that device current
            e = cudaGetSymbolAddress(&ws, g_static_workspace);
            if (e == cudaSuccess) g_static_ptr[dev].store(ws, std::memory_order_relaxed);
        }
    }
    if (e != cudaSuccess) {
        g_last_cuda_error = int(e);
        (void)cudaGetLastError();
        return EQUARX_ERR_CUDA;
    }
    // (the range call repeats the table checks, now including overlap with the built-in workspace)
    return equarx_allreduce_sim_range(in_bf16, out_bf16, nranks, count, block, ws,
                                      size_t(EQUARX_STATIC_WORKSPACE_BYTES), 0, 0, nranks, stream);
}

}  // extern "C"
