/*
 * equarx.h -- C ABI of the B200 (sm_100a) library for the arithmetic hot path
 * of EQuARX (arXiv 2506.17615): dynamic block-wise int8 quantization and the
 * dequantize / fp32-accumulate / requantize work that runs beside the steps
 * of a ring AllReduce, simulated on ONE GPU over N logical ranks whose bf16
 * buffers all live in that GPU's memory.  equarx_ring_allreduce, at the end,
 * is the same arithmetic as a ring with one rank per device.
 *
 * Conventions for every function
 *   - extern "C"; returns an EQUARX_* status; never throws, aborts or exits.
 *   - Arguments are validated on the host first; on a validation error
 *     nothing is launched and no CUDA call is made.
 *   - A failing launch is reported as EQUARX_ERR_CUDA (the CUDA error code is kept for
 *     equarx_last_cuda_error()); the launches that preceded it in the same call stay
 *     enqueued.  For tests, EQUARX_INJECT_LAUNCH_ERROR=<code> in the environment makes
 *     every launch report that code without launching anything.
 *   - Work is enqueued on `stream` and the call returns without
 *     synchronising.  The per-step calls, equarx_allreduce_sim(_range),
 *     equarx_allreduce_sim_pipelined, equarx_allreduce_sim_flavour and
 *     equarx_allreduce_sim_bf16 only enqueue kernel launches (and one memset for a
 *     flavour trace), so they can be recorded by stream capture and replayed as a
 *     CUDA graph; for messages below a few MB per rank, where launch and call
 *     overhead dominate, a replay takes about half the time of the direct calls.
 *   - Device buffers must stay valid until the stream has reached the work.
 *     The library allocates and frees nothing: the caller owns every buffer,
 *     including the workspace.
 *   - Pointer tables (`in_bf16`, `out_bf16`) are HOST arrays of DEVICE
 *     pointers; they are copied into kernel parameters during the call and
 *     may be freed as soon as it returns.  All other pointers are DEVICE
 *     pointers.
 *   - bf16 tensors are raw 16-bit words; bf16 buffers must be 32-byte
 *     aligned (they are moved with 256-bit accesses) and so must workspaces;
 *     int8 code buffers 16-byte aligned, scale buffers 4-byte aligned.
 *   - `block` is the number of contiguous elements that share one fp32
 *     scale (Section 3.2, Fig. 3: one scale factor per block of entries);
 *     supported values 64, 128, 256, 512.
 *   - Inputs must be finite, and so must every fp32 partial sum along a
 *     chain (|sum| below the fp32 maximum).  Inf/NaN inputs and overflowing
 *     sums are outside the contract: no trap, result unspecified.
 *
 * Arithmetic (identical, bit for bit, in every entry point)
 *   amax  = max |v| over the block                      (Section 3.2, max reduction)
 *   scale = amax / 127, inv = 127 / amax (IEEE fp32);   both 0 if amax < 2^-118
 *   code  = rne(v * inv) in [-127, 127]                 (symmetric int8, Section 4)
 *   hop   : v = fma((float)code, scale, (float)local)   (Section 3.1: dequantize to
 *           FP32, add the local counterpart), then quantize v again
 *   final : out = bf16_rne((float)code * scale)         (Section 3.4)
 */
#ifndef EQUARX_H_
#define EQUARX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Same type as cudaStream_t (which is `struct CUstream_st *`). */
typedef struct CUstream_st *equarx_stream_t;

#define EQUARX_MAX_RANKS 64

enum equarx_status {
    EQUARX_OK = 0,
    EQUARX_ERR_NULL = 1,       /* a required pointer (or table entry) is NULL            */
    EQUARX_ERR_NRANKS = 2,     /* nranks < 1 or > EQUARX_MAX_RANKS                       */
    EQUARX_ERR_BLOCK = 3,      /* block not in {64, 128, 256, 512}                       */
    EQUARX_ERR_COUNT = 4,      /* count 0, not a multiple of block (per-step calls) or
                                  of nranks*block (simulations), or above 2^40           */
    EQUARX_ERR_ALIGN = 5,      /* a pointer breaks the alignment rules above             */
    EQUARX_ERR_WORKSPACE = 6,  /* workspace_bytes smaller than *_workspace_bytes()       */
    EQUARX_ERR_ALIAS = 7,      /* buffers overlap in a way the call does not allow       */
    EQUARX_ERR_CUDA = 8,       /* a launch failed; see equarx_last_cuda_error()          */
    EQUARX_ERR_STATIC_LIMIT = 9, /* problem too large for the built-in workspace of
                                  equarx_allreduce_sim_static                            */
    EQUARX_ERR_FLAVOUR = 10    /* flavour is not a combination of EQUARX_FLAVOUR_* bits  */
};

/*
 * Ring step 0 (Section 3.1): the shard a rank sends first is quantized; what
 * travels is the int8 payload together with its scale factors.  The paper's two
 * phases (Q_p1 finds the metadata, Q_p2 scales the data) are one pass over
 * registers here.
 *   x_bf16 : count bf16 words (device, read)
 *   codes  : count int8 (device, written)
 *   scales : count/block fp32 (device, written); scales[b] belongs to
 *            elements [b*block, (b+1)*block)
 * count must be a multiple of block.
 */
int equarx_quantize_blocks(const void *x_bf16, size_t count, int block,
                           int8_t *codes, float *scales, equarx_stream_t stream);

/*
 * Ring steps 1..N-1 (Section 3.1): the received shard is widened to fp32 and
 * added to this rank's counterpart, and the partial sum is quantized again for
 * the next hop.  The fp32 partial sum lives in registers only.
 *   codes_in, scales_in   : the received message (device, read)
 *   local_bf16            : this rank's counterpart shard, count bf16 (device, read)
 *   codes_out, scales_out : the message for the next hop (device, written);
 *                           must not overlap the received message
 */
int equarx_rs_step_dequant_add_requant(const int8_t *codes_in, const float *scales_in,
                                       const void *local_bf16, size_t count, int block,
                                       int8_t *codes_out, float *scales_out,
                                       equarx_stream_t stream);

/*
 * Receive side of the quantized all-gather (Section 3.4: the extra
 * quantize/dequantize pair; its quantize half is the requantization of the
 * last reduce-scatter step).
 *   out_bf16 : count bf16 words (device, written)
 */
int equarx_ag_dequant(const int8_t *codes, const float *scales, size_t count, int block,
                      void *out_bf16, equarx_stream_t stream);

/*
 * Bytes of workspace equarx_allreduce_sim needs; 0 if the arguments are
 * invalid.  The workspace holds messages.  A message (one shard's codes and
 * scales) is stored as a sequence of 544-byte records, one per tile of 512
 * consecutive elements of the shard: first 8 floats of metadata (the tile's
 * 512/block scales in order, then zeros), then the tile's 512 int8 codes
 * (metadata ahead of the payload it describes, the order Section 3.1 sends them in).  The last record
 * of a message is only partly used if the shard is not a multiple of 512.
 * A message slot is tiles = ceil(shard/512) records; slot i starts at byte
 * i*tiles*544.  "Event j of shard k" is the message sent at ring step j by rank
 * (k+1+j) mod nranks; event nranks-1 is the all-gather message.  Without trace
 * there are 2*nranks slots and the event's slot is 2*k + (j&1) (ping-pong per
 * shard: on return the workspace holds the last two events of every shard).
 * With trace there are nranks*nranks slots, the event's slot is k*nranks + j
 * and every message of the run is kept.
 */
size_t equarx_allreduce_sim_workspace_bytes(int nranks, size_t count, int block, int keep_trace);

/*
 * The whole simulated quantized AllReduce: full-loop ring reduce-scatter
 * (Section 3, Fig. 1; adder chain of Section 3.3, Fig. 4) followed by the
 * quantized all-gather (Section 3.4), as nranks+1 launches on `stream`:
 * step 0 quantizes, steps 1..nranks-1 dequantize-add-requantize, the last
 * launch dequantizes every reduced shard into all nranks outputs.  Rank r
 * sends to rank (r+1) mod nranks; at step s it sends shard (r-1-s) mod nranks;
 * shard k is finished on rank k.
 *   in_bf16[r]  : count bf16 words of rank r (device, read)
 *   out_bf16[r] : count bf16 words (device, written); out_bf16[r] == in_bf16[r]
 *                 is allowed (in place); any other overlap between buffers is
 *                 rejected with EQUARX_ERR_ALIAS
 *   workspace   : equarx_allreduce_sim_workspace_bytes() bytes (device), not
 *                 overlapping any input or output; contents on return are the
 *                 messages as laid out above
 * count (per rank) must be a multiple of nranks*block.
 */
int equarx_allreduce_sim(const void *const *in_bf16, void *const *out_bf16,
                         int nranks, size_t count, int block,
                         void *workspace, size_t workspace_bytes, int keep_trace,
                         equarx_stream_t stream);

/*
 * The same schedule, restricted to launches first_launch..last_launch
 * (inclusive) of the nranks+1 launches: launch 0 is ring step 0 (quantize),
 * launch s in 1..nranks-1 is ring step s (dequantize-add-requantize on every
 * rank), launch nranks is the all-gather dequantize.  Running the ranges
 * [0,a], [a+1,b], ... [.., nranks] in order on one stream gives exactly
 * equarx_allreduce_sim; a profiler or a bench can bracket single steps this
 * way.  Requires 0 <= first_launch <= last_launch <= nranks, else
 * EQUARX_ERR_COUNT.  Other arguments as for equarx_allreduce_sim.
 */
int equarx_allreduce_sim_range(const void *const *in_bf16, void *const *out_bf16,
                               int nranks, size_t count, int block,
                               void *workspace, size_t workspace_bytes, int keep_trace,
                               int first_launch, int last_launch, equarx_stream_t stream);

/*
 * The same AllReduce as ONE persistent launch.  Section 3.1 splits a shard into
 * microshards that move through the ring steps independently of one another;
 * here a microshard is a tile of 512 elements and one warp carries it through
 * all nranks steps and the all-gather without waiting for the rest of the
 * shard.  Outputs, and with keep_trace the whole trace, are identical to
 * equarx_allreduce_sim bit for bit; only the order in which tiles advance
 * differs.  Two forms:
 *
 *   keep_trace != 0 (deep-pipelined, every message materialised): each hop
 *     message is written to memory as a record and read back from there by the
 *     neighbouring lane, which acts for the receiving rank.  The workspace
 *     receives the trace exactly as equarx_allreduce_sim lays it out.
 *   keep_trace == 0 (chain-fused): the adder chain of a tile (Section 3.3,
 *     Fig. 4) depends on no other tile, so the lane that quantized a group for
 *     the sending rank continues as the receiving rank; the message (int8 code
 *     values and the block scale) stays in registers and is never stored.  The
 *     kernel reads every bf16 input once and writes every bf16 output once:
 *     4 bytes of memory traffic per element of every rank, which is the
 *     roofline of this form; the hop messages of the ring schedule
 *     (2 + 8/block more bytes per element) are not moved at all.  The workspace
 *     is not touched; EQUARX_PIPELINE_MIN_WORKSPACE_BYTES is a token size so that
 *     one allocation pattern serves both forms.
 *
 * All other arguments and rules as for equarx_allreduce_sim.
 */
#define EQUARX_PIPELINE_MIN_WORKSPACE_BYTES 32u
size_t equarx_allreduce_sim_pipelined_workspace_bytes(int nranks, size_t count, int block, int keep_trace);
int equarx_allreduce_sim_pipelined(const void *const *in_bf16, void *const *out_bf16,
                                   int nranks, size_t count, int block,
                                   void *workspace, size_t workspace_bytes, int keep_trace,
                                   equarx_stream_t stream);

/*
 * equarx_allreduce_sim_pipelined with keep_trace = 0 for a call that does NOT depend on
 * earlier work of `stream` that may still be running.  By calling it the caller vouches
 * that no such unfinished work writes any in_bf16[r] or reads or writes any out_bf16[r]
 * (typically: the earlier work is AllReduces of this library on other tensors).  The
 * kernel then starts while that work is still finishing instead of waiting for it,
 * which removes the idle gap between back-to-back launches (measured on B200: 37.4
 * instead of 41.9 us for 8 x 15.7 MB, 211.7 instead of 220.4 us for 8 x 88 MB), and it
 * waits for that work only before it exits, so everything enqueued AFTER this call
 * still finds all earlier work of the stream complete.  Same arguments, rules and
 * results as equarx_allreduce_sim_pipelined; no workspace is needed.
 */
int equarx_allreduce_sim_pipelined_unordered(const void *const *in_bf16, void *const *out_bf16,
                                             int nranks, size_t count, int block,
                                             equarx_stream_t stream);

/*
 * The AllReduce of equarx_allreduce_sim_pipelined (keep_trace = 0) for tensors
 * that live in HOST memory: what Section 3.1 and Section 3.4 compute, with the
 * copies to and from the device issued by this call.
 *   host_in[r]  : count bf16 words of rank r in host memory (read).  Pinned
 *                 (page-locked) memory makes the copies asynchronous; pageable
 *                 memory works and makes the call block for the copies.
 *   host_out[r] : count bf16 words in host memory (written); may equal
 *                 host_in[r].
 *   staging     : DEVICE memory supplied by the caller,
 *                 equarx_allreduce_sim_host_staging_bytes(nranks, count) bytes
 *                 (2 * count * nranks), 32-byte aligned; holds the nranks
 *                 tensors on the device and is reduced in place.
 * The call enqueues on `stream`: nranks host-to-device copies (one plain
 * cudaMemcpyAsync per rank tensor), the kernel, nranks device-to-host copies, and
 * returns without synchronising; host_out is valid once the stream has reached the
 * last copy.  The library still allocates nothing.  A failing copy is reported as
 * EQUARX_ERR_CUDA like a failing launch.  Two calls on two streams with two
 * staging buffers overlap each other's copies and kernels.
 */
size_t equarx_allreduce_sim_host_staging_bytes(int nranks, size_t count);
int equarx_allreduce_sim_host(const void *const *host_in, void *const *host_out,
                              int nranks, size_t count, int block,
                              void *staging, size_t staging_bytes,
                              equarx_stream_t stream);

/*
 * The other flavours of the method, in the deep-pipelined form of
 * equarx_allreduce_sim_pipelined (one persistent launch, one warp per
 * 512-element tile).  `flavour` is a combination of:
 *   EQUARX_FLAVOUR_SEMI_LOOP : semi-loop ring (Section 3.3, Fig. 5): shard k is
 *       reduced by two half chains that meet at its owner,
 *       A: k+N/2 -> k+N/2-1 -> ... -> k+1 -> k and B: k+N/2+1 -> ... -> k-1 -> k
 *       (on 4 devices 2 -> 1 -> 0 and 3 -> 0, the paper's example); the owner
 *       adds B's partial, then A's.  nranks must be even.  Without this bit:
 *       the full-loop chain k+1 -> k+2 -> ... -> k.
 *   EQUARX_FLAVOUR_QUANT_RS  : the reduce-scatter hops carry int8 records
 *       (Section 3.1); without it they carry bf16 and every add is rounded to
 *       bf16, as in the BF16 baseline.
 *   EQUARX_FLAVOUR_QUANT_AG  : the reduced shard takes one more
 *       quantize/dequantize pair (Section 3.4); without it the owner's sum is
 *       rounded to bf16 and forwarded as is.
 *   EQUARX_FLAVOUR_E4M3, EQUARX_FLAVOUR_E5M2 (at most one, and only with a
 *       quantized stage): the payload is FP8 instead of int8 (Section 4 names
 *       all three).  Same rule with the format's largest finite value in place
 *       of 127: scale = amax/448 (E4M3, bias 7, no infinities) or amax/57344
 *       (E5M2, bias 15), code = fp8_rne(v * (FMAX/amax)) saturating at +-FMAX;
 *       blocks with amax < 2^-117 (E4M3) or 2^-110 (E5M2) get scale 0 and zero
 *       codes.  FP8 has a negative zero, so a flushed negative input comes back
 *       as -0.0.  The codes of a trace are the raw FP8 bytes.
 * QUANT_RS | QUANT_AG is equarx_allreduce_sim_pipelined's result bit for bit;
 * 0 is the unquantized ring of equarx_allreduce_sim_bf16.
 * Like equarx_allreduce_sim_pipelined the call has two forms.  Without
 * keep_trace every message stays in the registers of the lane that produced it
 * (chain-fused; for flavour 0 this is the unquantized comparator in the same
 * form as the quantized single launch) and the workspace, of the token size
 * EQUARX_PIPELINE_MIN_WORKSPACE_BYTES, is not touched.  With keep_trace every
 * message goes through memory and the workspace is EQUARX_FLAVOUR_FIFO_BYTES of
 * staging space followed by a trace laid out as for equarx_allreduce_sim.
 * Events of a full loop: j = 0..N-2 the hops in chain order, N-1 the all-gather
 * message; of a semi loop: 0..N/2-1 chain A's hops, N/2..N-2 chain B's hops, N-1
 * the all-gather message.  Events that the flavour does not quantize are zeroed.
 * Other arguments and rules as for equarx_allreduce_sim.
 */
#define EQUARX_FLAVOUR_SEMI_LOOP 1
#define EQUARX_FLAVOUR_QUANT_RS 2
#define EQUARX_FLAVOUR_QUANT_AG 4
#define EQUARX_FLAVOUR_E4M3 8
#define EQUARX_FLAVOUR_E5M2 16
#define EQUARX_FLAVOUR_FIFO_BYTES (16u * 1024u * 1024u)
size_t equarx_allreduce_sim_flavour_workspace_bytes(int nranks, size_t count, int block, int flavour,
                                                    int keep_trace);
int equarx_allreduce_sim_flavour(const void *const *in_bf16, void *const *out_bf16,
                                 int nranks, size_t count, int block, int flavour,
                                 void *workspace, size_t workspace_bytes, int keep_trace,
                                 equarx_stream_t stream);

/* Workspace bytes of the unquantized comparator (two generations of bf16 messages: 4*count); 0 if invalid. */
size_t equarx_allreduce_sim_bf16_workspace_bytes(int nranks, size_t count);

/*
 * Unquantized comparator (the "baseline BF16 AllReduce" of Section 4): the
 * same ring with bf16 messages, p = bf16_rne((float)p_in + (float)local) at
 * every hop.  Step 0 sends the raw shard, so the first hop reads its
 * neighbour's input directly; nranks launches (nranks-1 hops + all-gather).
 * count must be a multiple of 16*nranks.  Same aliasing rules as above.
 */
int equarx_allreduce_sim_bf16(const void *const *in_bf16, void *const *out_bf16,
                              int nranks, size_t count,
                              void *workspace, size_t workspace_bytes,
                              equarx_stream_t stream);

/*
 * equarx_allreduce_sim without a caller-provided workspace.  (The paper has no
 * counterpart for this entry point; it exists for the callers described here.)
 *
 * Who it is for: code that must run the simulation but is not in a position to
 * hand over scratch memory -- a plugin inside a host application that owns the
 * whole device heap, a serving loop whose memory plan is frozen after start-up,
 * a process that is not permitted to call cudaMalloc at all.  Such callers still
 * own their input and output tensors; what they lack is a place for the hop
 * messages.  This function keeps that place inside the library: a fixed array of
 * EQUARX_STATIC_WORKSPACE_BYTES bytes in the library's device image.  Every GPU
 * on which the library is loaded carries that array until the process exits,
 * whether this function is ever called or not.
 *
 * It calls no cudaMalloc, cudaFree or other allocating routine.  The result is
 * bit-identical to equarx_allreduce_sim (keep_trace = 0) on the same inputs.
 *
 * Limits and rules
 *   - The problem must fit: equarx_allreduce_sim_workspace_bytes(nranks, count,
 *     block, 0) <= EQUARX_STATIC_WORKSPACE_BYTES, else EQUARX_ERR_STATIC_LIMIT
 *     and nothing is launched.  (16 MiB holds, for example, 8 ranks x 7.86 M
 *     elements: 2*8 message slots of 1920 records.)
 *   - The first call on a given device looks up the array's device address
 *     (cudaGetSymbolAddress, with that device current) and remembers it.  Make
 *     that first call during normal execution, before any stream capture
 *     begins on that device.
 *   - All calls on a device share the one array.  Two calls whose kernels can
 *     run at the same time (different streams, no ordering between them) race
 *     on it and produce garbage; order them yourself.  The array keeps the
 *     previous call's messages; nothing in it has to start at zero, because
 *     every message is written by an earlier launch of the same call before it
 *     is read.
 *   - Arguments, aliasing rules and the other error codes are those of
 *     equarx_allreduce_sim.
 */
#define EQUARX_STATIC_WORKSPACE_BYTES (16u * 1024u * 1024u)
int equarx_allreduce_sim_static(const void *const *in_bf16, void *const *out_bf16,
                                int nranks, size_t count, int block,
                                equarx_stream_t stream);

/*
 * The quantized ring AllReduce with one rank per device: the setting of Section 3
 * (Fig. 1) and Section 3.1 (Fig. 2: metadata first, microshards pipelined so that
 * transfers overlap the dequantize / add / quantize work).  Each rank runs ONE
 * persistent kernel that performs all nranks ring steps and the all-gather.  A
 * microshard is a tile of 512 elements and its message one 544-byte record (layout as
 * for equarx_allreduce_sim).  The sending rank stores the record directly into the
 * RECEIVING rank's mailbox (peer memory: NVLink when the ranks are on different GPUs)
 * and then releases a per-tile flag; the receiving warp polls that flag.  The last
 * reduce-scatter step stores the all-gather message of the rank's own shard into every
 * rank's mailbox, and every rank dequantizes the nranks messages it received.  Ring
 * direction, shard order and arithmetic are those of equarx_allreduce_sim, so the
 * outputs and every message are identical to it bit for bit.
 *
 * A call hosts the consecutive ranks rank_first .. rank_first + ranks_here - 1 on the
 * current device, in one cooperative launch (all its CTAs are resident at once).
 * ranks_here = 1 is the multi-GPU case: one process and one call per GPU, all with
 * the same epoch.  ranks_here = nranks runs the whole ring on a single GPU.
 *
 *   in_bf16[i], out_bf16[i] : HOST arrays of ranks_here DEVICE pointers: tensors of
 *                 rank rank_first + i (count bf16 words each; out may equal in)
 *   mailboxes   : HOST array of nranks DEVICE-addressable pointers, mailbox of every
 *                 rank of the ring, own ranks included; a peer's mailbox is its
 *                 allocation mapped into this process (CUDA IPC or any other
 *                 peer mapping).  Each is equarx_ring_mailbox_bytes() bytes, 32-byte
 *                 aligned, and must be zeroed ONCE before its first use.
 *                 Layout: slots 0..nranks-2 hold the message received at ring step
 *                 slot+1, slots nranks-1..2*nranks-2 the all-gather message of shard
 *                 slot-(nranks-1); a slot is ceil(count/nranks/512) records; then one
 *                 uint32 flag per (slot, tile), slot-major.
 *   epoch       : >= 1, the same on every rank of one AllReduce, and larger than in
 *                 any earlier call that used these mailboxes (a flag equal to the
 *                 epoch marks a complete record, so nothing is cleared between calls).
 *                 Calls that share mailboxes must be ordered on each rank's stream.
 *   timeout_ns  : longest wait for one message; 0 selects 1 second.  A wait that runs
 *                 out, or that sees another warp's failure, makes the warp record
 *                 {epoch, rank, step, tile} in `status` (first failure of the call
 *                 only) and leave; the kernel always terminates, never traps.  step is
 *                 the ring step, or nranks + shard for an all-gather message.
 *   status      : DEVICE memory, 4 x uint32, 16-byte aligned, zeroed ONCE by the caller
 *                 before its first use (like the mailboxes); nothing clears it between
 *                 calls.  Read it after synchronising: status[0] equal to the call's
 *                 epoch means that call timed out, any other value that every
 *                 message of the call arrived.
 * Returns EQUARX_ERR_CUDA if the cooperative launch is refused (for example more hosted
 * ranks than CTAs that fit on the device).
 * Not exercised on more than one GPU; the ranks_here = nranks form is what the tests run.
 */
size_t equarx_ring_mailbox_bytes(int nranks, size_t count, int block);
int equarx_ring_allreduce(const void *const *in_bf16, void *const *out_bf16,
                          int rank_first, int ranks_here, int nranks, size_t count, int block,
                          void *const *mailboxes, uint32_t epoch, uint64_t timeout_ns,
                          uint32_t *status, equarx_stream_t stream);

/* Static, human-readable name of a status. */
const char *equarx_status_string(int status);

/* The cudaError_t (as int) behind the calling thread's last EQUARX_ERR_CUDA, else 0. */
int equarx_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* EQUARX_H_ */
