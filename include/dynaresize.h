/*
 * dynaresize.h -- C ABI of the per-GPU role-switch state transform for sm_100a (B200).
 *
 * When runtime GPU reallocation turns a Training GPU into a Rollout GPU (or back), the GPU has to drop
 * the state of its old role and take in the weights and optimizer state of the new one (paper Sec. 1,
 * challenge 2), i.e. bring in whatever state the new topology asks for (Sec. 3.3).  This library is
 * that per-GPU step:
 *
 *   Training -> Rollout : read the FSDP-style flat fp32 master buffer, un-flatten it, fuse Q/K/V and
 *                         gate/up, slice for a tensor-parallel degree and rank, cast to bf16
 *                         (round to nearest, ties to even) into a contiguous rollout arena;
 *   Rollout -> Training : the inverse layout map (bf16 widened exactly to fp32);
 *   both directions     : stream optimizer state (fp32 master, Adam m, Adam v) to and from host
 *                         memory in fixed chunks through a bounded pinned ring (the chunk-wise
 *                         streaming through host buffers of Sec. 3.3), weights first
 *                         on the way back (the deferred optimizer reload of Sec. 3.3).
 *
 * Conventions
 *   - Every function returns an int status: DR_OK (0) or a negative dr_status.  Nothing throws,
 *     aborts or exits.  dr_last_error() gives a thread-local detail string for the last failure.
 *   - "dev" pointers are CUDA device pointers of the current device; "host" pointers are ordinary
 *     host pointers.  The caller owns every buffer it passes.  A plan owns only its device segment
 *     table, its pinned staging ring and two internal streams.
 *   - Streams and events are passed as void* holding a cudaStream_t / cudaEvent_t (NULL stream =
 *     the legacy default stream).
 *   - Stream ordering.  dr_reshard, dr_reshard_inverse, dr_reshard_groups and dr_reshard_static run on
 *     the stream they are given and need nothing more.  dr_stage_out, dr_stage_in and
 *     dr_reshard_stream copy on streams the plan owns (created non-blocking, so not even the legacy
 *     default stream orders them).  On entry they therefore make their streams wait for everything
 *     already enqueued on desc->caller_stream (or, when desc->wait_event is set, for that event
 *     alone), so that device buffers the caller has just filled, zeroed or freed-and-reallocated on
 *     that stream are ready before the first copy touches them.  Work the caller has pending on any
 *     OTHER stream that touches those buffers must be covered by wait_event or a synchronise.  The
 *     three calls block until all of their copies and kernels have completed, so whatever the caller
 *     enqueues after they return, on any stream, sees the result; done_event is recorded for callers
 *     that hand the ordering to a third stream.  None of the three may be called while caller_stream
 *     is being captured into a CUDA graph.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with DR_ERR_CUDA.
 *   - Matrices are [out_features, in_features], row-major.
 */
#ifndef DYNARESIZE_H
#define DYNARESIZE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DR_VERSION 1u
#define DR_MAX_STAGE_BUFS 8u

typedef enum dr_status {
    DR_OK = 0,
    DR_ERR_INVALID = -1,     /* NULL pointer, bad struct_size/version, value out of range          */
    DR_ERR_UNSUPPORTED = -2, /* shapes not divisible by tp, moe_tp != 1, unknown kind/dtype         */
    DR_ERR_SIZE = -3,        /* a buffer is smaller than the plan needs                             */
    DR_ERR_ALIGN = -4,       /* a base pointer is not 16-byte aligned                               */
    DR_ERR_NOMEM = -5,       /* host, pinned or device allocation failed                            */
    DR_ERR_CUDA = -6,        /* a CUDA runtime call failed (detail in dr_last_error)                */
    DR_ERR_BUDGET = -7,      /* staging budget cannot hold two chunk slots                          */
    DR_ERR_SINK = -8,        /* the chunk callback returned non-zero                                */
    DR_ERR_TIMEOUT = -9,     /* a bounded host-side wait ran out                                    */
    DR_ERR_STATE = -10       /* call not valid for this plan (e.g. reshard on a host-only plan)     */
} dr_status;

enum { DR_SRC_FSDP_FLAT = 1 };
enum { DR_DST_ROLLOUT_FUSED = 1 };
enum { DR_F32 = 1, DR_BF16 = 2, DR_FP8_E4M3_B128 = 3 };

/* Decoder shape.  Dense when n_experts == 0 (SwiGLU of width ffn), else every layer holds a router
 * [n_experts, hidden] and n_experts SwiGLU experts of width moe_ffn (ffn is ignored). */
typedef struct dr_model_spec {
    uint32_t struct_size, version; /* sizeof(dr_model_spec), DR_VERSION */
    uint32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    uint32_t n_experts, moe_ffn;
    uint8_t tied_embeddings; /* 1: no separate lm_head; the rollout lm_head aliases embed            */
    uint8_t qk_norm;         /* 1: per-layer q_norm[head_dim], k_norm[head_dim] vectors exist        */
    uint8_t pad[2];
} dr_model_spec;

/* Training-side layout: all parameters flattened in canonical order
 *   embed; per layer: in_norm, q, k, v, (q_norm, k_norm), o, post_norm,
 *   dense: gate, up, down | MoE: router, then per expert gate_e, up_e, down_e;
 *   final_norm; lm_head unless tied
 * each starting at a multiple of align_elems; N elements in all, S = ceil(N / world) per rank.
 * gathered = 1: the source buffer holds world * S elements (the whole flat buffer);
 * gathered = 0: it holds rank `rank`'s S elements only, and only elements inside that shard move. */
typedef struct dr_src_layout {
    uint32_t struct_size, kind /* DR_SRC_FSDP_FLAT */, dtype /* DR_F32 */;
    uint32_t world, rank, gathered, align_elems /* >= 1 */;
} dr_src_layout;

/* Rollout-side layout at (tp, rank): tensors in arena order, each start aligned to arena_align_bytes:
 *   embed rows of this rank; per layer: in_norm, qkv = [q_t; k_t; v_t], (q_norm, k_norm),
 *   o columns of this rank, post_norm, dense: gate_up = [gate_t; up_t], down columns of this rank |
 *   MoE: router, w13[e] = [gate_e; up_e] for every expert, w2[e] = down_e;
 *   final_norm; lm_head rows of this rank (an alias of embed when tied).
 * Norms and the router are replicated on every rank; by default experts are neither sliced nor
 * dropped.  The optional fields select the variants rollout engines use (kv-head replication,
 * vocabulary padding, expert tensor / expert parallelism). */
typedef struct dr_dst_layout {
    uint32_t struct_size, kind /* DR_DST_ROLLOUT_FUSED */, dtype /* DR_BF16 or DR_F32 */;
    uint32_t moe_tp;            /* 1: experts unsliced; == tp: expert FFN width sliced like the dense MLP
                                   (gate_e / up_e rows, down_e columns of this rank)                     */
    uint32_t arena_align_bytes; /* power of two >= 16, e.g. 256                                          */
    uint32_t kv_replicate;      /* 1: tp may be a multiple of n_kv_heads; rank t then holds the single kv
                                   head t / (tp / n_kv_heads) (each head on tp / n_kv_heads ranks)       */
    uint32_t vocab_pad;         /* > 0: embed / lm_head are padded to a multiple of this many rows before
                                   slicing; padding rows occupy the arena but are never written or read  */
    uint32_t moe_ep;            /* expert parallel degree (0 or 1: all experts); must divide n_experts   */
    uint32_t moe_ep_rank;       /* this rank keeps experts [rank * E / ep, (rank + 1) * E / ep)           */
} dr_dst_layout;

/*
 * dtype DR_FP8_E4M3_B128 (a rollout-engine layout, no counterpart in the paper): the linear weights
 * (qkv, o, gate_up, down, w13, w2) are written as fp8 e4m3 with one fp32 scale per 128 x 128 block of
 * the rollout tensor; embed, lm_head, router and the norms stay bf16.  Per block: amax = max |x| (NaNs
 * skipped), stored scale = amax / 448 in fp32, held inside [2^-126, FLT_MAX] (so a block whose
 * amax / 448 underflows, the all-zero block included, keeps zeros as zeros and yields no NaN, and a block
 * holding an infinity keeps a finite scale); code = e4m3(x / scale): one fp32 division rounded to
 * nearest, then round to nearest even onto the e4m3 grid, magnitudes above 448 saturating to 448,
 * NaN -> 0x7F.  A consumer dequantises with code * scale.  A quantised tensor occupies rows * cols
 * bytes at arena_off, then its scales, row-major, at scale_off (the next multiple of
 * arena_align_bytes).  Needs the whole flat buffer (gathered = 1 or world = 1): a block cannot be
 * scaled from part of its elements.
 * Supported on such a plan: dr_reshard, dr_reshard_groups, and dr_reshard_inverse, which writes
 * value(code) * scale (one fp32 multiplication; any NaN becomes 0x7FC00000) to the flat positions of
 * the quantised tensors and widens the bf16 ones.  dr_reshard_static, dr_reshard_stream,
 * dr_reshard_push, dr_plan_ranges and dr_plan_window_host return DR_ERR_UNSUPPORTED.
 */
typedef struct dr_plan dr_plan;

typedef struct dr_plan_info {
    uint64_t flat_elems;      /* N                                                                   */
    uint64_t shard_elems;     /* S                                                                   */
    uint64_t src_bytes;       /* bytes the source (flat) buffer must hold: 4*W*S or 4*S              */
    uint64_t dst_bytes;       /* bytes the rollout arena must hold                                   */
    uint64_t n_tensors;       /* rollout tensors (aliases included)                                  */
    uint64_t n_segments;      /* entries of the device segment table                                 */
    uint64_t n_tiles;         /* work tiles one launch processes                                     */
    uint64_t elems_moved;     /* elements one dr_reshard / dr_reshard_inverse moves                  */
    uint64_t bytes_moved_fwd; /* algorithmic bytes of dr_reshard: (4 + dst element size) * elems     */
    uint64_t bytes_moved_inv; /* the same for dr_reshard_inverse                                     */
    uint64_t quant_elems;     /* DR_FP8_E4M3_B128 plans: elements written as fp8 (counted in elems_moved) */
    uint64_t quant_blocks;    /* and the number of 128 x 128 blocks, one fp32 scale each              */
    uint64_t n_groups;        /* n_layers + 2: embed, every layer, final norm with lm_head            */
    uint64_t bulk_forward;    /* 1: dr_reshard runs the kernel that brings tiles in with the TMA unit's
                                 bulk copies (plans of 2^28 elements or more with under 2 % of them in
                                 strided segments); 0: the kernel that moves them through registers.
                                 Same result.  The environment variable DR_FORWARD_KERNEL = bulk |
                                 register, read when a plan is created, overrides the choice.          */
} dr_plan_info;

typedef struct dr_tensor_desc {
    char name[64];
    uint64_t arena_off; /* byte offset of the tensor inside the rollout arena                       */
    uint64_t rows, cols;
    int64_t alias_of;   /* >= 0: index of the rollout tensor whose storage this one shares           */
    uint32_t elem_size; /* bytes per element of the payload: 4, 2, or 1 (fp8)                         */
    uint32_t quantised; /* 1: fp8 payload with block scales                                          */
    uint64_t scale_off; /* quantised: byte offset of the fp32 scales [scale_rows, scale_cols]         */
    uint64_t scale_rows, scale_cols; /* ceil(rows / 128), ceil(cols / 128)                            */
} dr_tensor_desc;

/* One entry of the compiled map: rows x row_len elements, row i read from source element
 * src_off + i * src_row_stride and written at arena byte dst_off + i * dst_row_stride * elem size.
 * Exposed so that the planner can be checked without a GPU. */
typedef struct dr_segment_desc {
    uint64_t dst_off;  /* bytes, relative to the arena base                                         */
    uint64_t src_off;  /* elements, relative to the source buffer the call receives                 */
    uint64_t rows, row_len, src_row_stride, dst_row_stride; /* elements                              */
    uint32_t vector_bytes; /* 32 / 16: source access width the kernel may use; 0: scalar path        */
    uint32_t tensor;       /* rollout tensor its first element belongs to (merged runs span several)  */
} dr_segment_desc;

/*
 * dr_plan_create -- compile the un-flatten / fuse / slice map for (spec, src, dst, tp, rank) into a
 * segment table and upload it to the current device (one small H2D copy; synchronous).  This is the
 * metadata a resize prepares ahead of the switch (Sec. 3.2 applies the same idea to communicators).
 * Errors: DR_ERR_INVALID, DR_ERR_UNSUPPORTED (n_q_heads, ffn, the padded vocabulary or, without
 * kv_replicate, n_kv_heads not divisible by tp; moe_tp not 1 or tp; moe_ep not dividing n_experts),
 * DR_ERR_NOMEM, DR_ERR_CUDA.  *out is NULL on failure.
 */
int dr_plan_create(const dr_model_spec* spec, const dr_src_layout* src, const dr_dst_layout* dst, uint32_t tp,
                   uint32_t rank, dr_plan** out);

/* Same planner, no device work: the plan answers queries only; reshard and staging calls on it
 * return DR_ERR_STATE.  For checking the planner where no GPU exists. */
int dr_plan_create_host(const dr_model_spec* spec, const dr_src_layout* src, const dr_dst_layout* dst, uint32_t tp,
                        uint32_t rank, dr_plan** out);

/* The part of `plan` whose source elements lie in [src_elem_lo, src_elem_hi) of the buffer the plan reads,
 * as a host-only plan whose source buffer is that window alone (what one chunk of dr_reshard_stream
 * repacks).  For inspection and checks; not for fp8 plans (DR_ERR_UNSUPPORTED).  DR_ERR_INVALID if the
 * window is empty or leaves the source buffer. */
int dr_plan_window_host(const dr_plan* plan, uint64_t src_elem_lo, uint64_t src_elem_hi, dr_plan** out);

int dr_plan_query(const dr_plan* plan, dr_plan_info* out);
int dr_plan_tensor(const dr_plan* plan, uint32_t i, dr_tensor_desc* out);   /* DR_ERR_INVALID if i >= n_tensors  */
int dr_plan_segment(const dr_plan* plan, uint64_t i, dr_segment_desc* out); /* DR_ERR_INVALID if i >= n_segments */

/*
 * dr_reshard -- Training -> Rollout (Sec. 1 challenge 2: taking in the new role's weights).  Enqueues the
 * gather / cast kernel on cuda_stream and returns; nothing is synchronised.
 *   src_dev : fp32 flat buffer (whole, or this rank's shard when gathered = 0), read only
 *   dst_dev : rollout arena; only mapped elements are written, gaps and (for gathered = 0) elements
 *             whose source lies in another shard keep their bytes
 * Every rollout element is the bf16 round-to-nearest-even cast of its source element (NaN -> 0x7FFF;
 * subnormals are rounded, not flushed), or a bit copy when the plan's dst dtype is DR_F32.
 * Errors (all found before launch): DR_ERR_SIZE if src_bytes / dst_bytes are below the plan's
 * requirement, DR_ERR_ALIGN if a base pointer is not 16-byte aligned, DR_ERR_STATE, DR_ERR_CUDA.
 * Bases that are 32-byte aligned let the kernels (the fp8 one included) use 256-bit accesses; with
 * 16-byte aligned bases they fall back to 128-bit ones, same result.
 * The plan is not modified: concurrent calls on different streams are allowed.  The call only enqueues
 * kernels, so (after one ordinary call has loaded the module) it may be recorded into a CUDA graph by
 * stream capture and replayed; the same holds for dr_reshard_inverse.
 */
int dr_reshard(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* dst_dev, uint64_t dst_bytes,
               void* cuda_stream);

/*
 * dr_reshard_inverse -- Rollout -> Training (Sec. 3.3: bringing back the state the new topology
 * needs)..  Scatters the rollout arena back to the flat positions it was taken from, widening
 * bf16 to fp32 exactly (bits << 16).  Only positions covered by this TP rank (and, for gathered = 0,
 * lying in this shard) are written; padding and everything else keep their bytes.  On an fp8 plan the
 * quantised tensors come back as value(code) * scale.  Asynchronous on cuda_stream; same errors as
 * dr_reshard.
 */
int dr_reshard_inverse(const dr_plan* plan, const void* rollout_dev, uint64_t rollout_bytes, void* flat_dev,
                       uint64_t flat_bytes, void* cuda_stream);

/* A group of rollout tensors that can be repacked on its own: group 0 is embed, group l + 1 is layer l,
 * the last group holds final_norm and lm_head. */
typedef struct dr_group_desc {
    uint32_t first_tensor, n_tensors; /* rollout tensors [first_tensor, first_tensor + n_tensors)        */
    uint64_t elems;                   /* elements the group moves (0 when its sources lie in other shards) */
    uint64_t bytes_moved;             /* algorithmic bytes: (4 + rollout element size) * elems            */
} dr_group_desc;
int dr_plan_group(const dr_plan* plan, uint32_t g, dr_group_desc* out); /* DR_ERR_INVALID if g >= n_groups */

/*
 * dr_reshard_groups -- dr_reshard restricted to groups [first, first + count): one layer (or a few) at a
 * time, so that whatever follows the repack of a layer (handing it to the rollout engine, sending it to
 * other GPUs) can overlap the repack of the next ones; this is the switch split into the fine-grained,
 * overlappable operations Sec. 3.1 and 3.3 argue for.  Elements of other groups keep their bytes;
 * running every group once, in any order, gives exactly dr_reshard's result.  Same arguments and errors
 * as dr_reshard, plus DR_ERR_INVALID for a range outside the groups.  fp8 plans: a group's quantised tensors
 * are block-scaled by the same call.
 */
int dr_reshard_groups(const dr_plan* plan, uint32_t first, uint32_t count, const void* src_dev, uint64_t src_bytes,
                      void* dst_dev, uint64_t dst_bytes, void* cuda_stream);

/*
 * Exchange after the local repack (Sec. 3.2: the weight synchronisation between roles that follows a
 * switch).  With gathered = 0 every FSDP rank repacks only the rollout elements whose sources lie in its
 * own shard; a rollout rank then needs the pieces of all W training ranks.  The pieces are already cast
 * to bf16, so they cross the links at half the bytes of gathering fp32 first.
 *
 * dr_plan_ranges -- the arena byte ranges [off, off + bytes) that dr_reshard on this plan writes,
 * ascending and coalesced (touching ranges merged).  Host arithmetic only.  Over the W shard-local plans
 * of one (tp, rank) these ranges are pairwise disjoint and their union is the range set of the gathered
 * plan: they are the send / receive lists of an all-gather of the repacked pieces.  Writes at most
 * max_ranges entries to out (out may be NULL when max_ranges is 0) and always the full count to
 * *n_ranges.  Not for fp8 plans (DR_ERR_UNSUPPORTED).
 */
typedef struct dr_range {
    uint64_t off, bytes;
} dr_range;
int dr_plan_ranges(const dr_plan* plan, uint64_t max_ranges, dr_range* out, uint64_t* n_ranges);

/*
 * dr_reshard_push -- dr_reshard fused with the exchange: the same gather / cast kernel stores every
 * element it produces into n_dst rollout arenas instead of one, so that a training rank repacks its
 * shard and delivers the pieces to the rollout ranks in one pass over its master shard, with no packed
 * send buffer and no second kernel.  dst_dev[i] are device pointers this GPU can store to: its own
 * memory, or peers' arenas mapped into this process (CUDA IPC or any other peer mapping, peer access
 * enabled by the caller); plain peer stores over NVLink, no multicast of any kind.  Every arena gets
 * exactly the bytes dr_reshard would write (the plan's dr_plan_ranges); all else keeps its bytes.
 *   n_dst   : 1 .. DR_MAX_PUSH_DST
 *   dst_dev : n_dst arena base pointers, each 16-byte aligned and dst_bytes large
 * The kernel waits on nothing and signals nothing: a consumer on another GPU may read its arena only
 * after the pushing rank's stream has reached the point after this call (an event shared between the
 * processes, or a host-side barrier after a stream synchronise), which is the caller's to arrange.
 * Once all W ranks of one (tp, rank) have pushed, every arena holds the gathered plan's result.
 * Asynchronous on cuda_stream; errors as dr_reshard, plus DR_ERR_INVALID for a bad n_dst or a NULL
 * entry and DR_ERR_UNSUPPORTED for fp8 plans.
 */
#define DR_MAX_PUSH_DST 8u
int dr_reshard_push(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* const* dst_dev, uint32_t n_dst,
                    uint64_t dst_bytes, void* cuda_stream);

/*
 * dr_reshard_static -- dr_reshard for callers that must not allocate device memory.  (The paper has
 * no counterpart; this is a deployment aid.)
 *
 * Who needs it: a worker whose framework has already given the whole GPU to its own memory pool, so
 * that a cudaMalloc at switch time would fail or take the head-room the incoming state needs; and a
 * switch that overlaps staging copies with the repack, which a cudaMalloc or cudaFree would stall
 * because both synchronise the device.  `plan` may come from dr_plan_create_host (no device memory at
 * all) or from dr_plan_create.  The segment table, which dr_plan_create keeps in cudaMalloc'ed
 * memory, is instead copied on `cuda_stream` into a fixed table inside the library (1 MiB, 16 384
 * segments; every GPU that loads the library holds it until the process exits), and the same kernel
 * runs from there.  The call itself allocates nothing, on host or device.
 *
 * Same arguments, result and errors as dr_reshard, plus DR_ERR_SIZE when the plan has more than
 * 16 384 segments (dr_plan_query: n_segments).  Unlike dr_reshard the call is not purely an enqueue:
 * the table is uploaded from ordinary (pageable) host memory with cudaMemcpyAsync, which the driver may
 * stage and for which it may make the host wait until earlier work on cuda_stream has drained.  The
 * first call on each device also looks up the table's device address.  All calls share the one table
 * and it keeps the previous call's entries: each call rewrites the entries it uses, in stream order,
 * before its kernel reads them, so calls on one stream are safe back to back, while calls that can
 * overlap on the GPU (different streams, or different threads on different streams) race on the table
 * and must be ordered by the caller.
 */
int dr_reshard_static(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* dst_dev, uint64_t dst_bytes,
                      void* cuda_stream);

/* Chunk callback: stage-out hands chunk `chunk_idx` (bytes [stream_off, stream_off + n) of the
 * stream) in `pinned`; stage-in asks the callback to fill `pinned` with those bytes.  The pointer is
 * valid only during the call.  A non-zero return stops the transfer with DR_ERR_SINK. */
typedef int (*dr_chunk_fn)(void* user, uint64_t chunk_idx, uint64_t stream_off, void* pinned, uint64_t n);

/*
 * Staging descriptor.  The state buffers form one logical byte stream X = buf_0 | buf_1 | ... of B
 * bytes.  Stage-out cuts X into chunks of chunk_bytes (chunk k = X[k C, min((k+1) C, B)); a chunk
 * that straddles a buffer boundary is one chunk made of two copies) and delivers them in increasing
 * k.  Stage-in restores the buffers in `order` (weights first); each buffer is cut into pieces of at
 * most chunk_bytes, numbered consecutively in that order.
 * At most budget_bytes of pinned ring memory are held: slots = floor(budget / chunk) >= 2.
 * Where the bytes rest:
 *   callback   != NULL : every chunk goes to / comes from the callback (excludes the other two)
 *   relay_dev[i] != NULL (stage-out only): buffer i is copied straight on to relay_dev[i] through the
 *                        ring, the old-rank -> new-rank pipeline of Sec. 3.3, never resting on the host
 *   host_arena != NULL : every buffer without a relay target rests in the arena (arena[0, B) is the
 *                        stream image, or host_offset[i] with DR_STAGE_HOST_OFFSETS); a pinned arena is
 *                        copied to directly (still chunk by chunk), a pageable one through the ring by
 *                        worker threads
 * A pageable arena is served by worker threads behind the pump (ring slot -> arena on the way out, arena ->
 * ring slot on the way in, in tasks of 1 MiB), so several chunks are in flight on the host side as well.
 * There are min(16, cores - 2) workers (two cores stay free for the pump and the driver's thread; the
 * environment variable DR_COPY_THREADS = 1..64, read when a plan first stages, overrides the count).
 * For such an arena a small ring is the fast one: about eight slots of 4 - 8 MiB stay in the host's
 * last-level cache, so a chunk is copied out right behind the DMA that delivered it (and filled right
 * before the DMA that reads it) without a round trip through host DRAM; measured 0.88 - 0.97 of the link
 * against 0.70 - 0.88 with slots of 256 MiB - 1 GiB (a relay reaches what the link gives with both
 * directions busy through the small ring on every box measured, through large slots only on some).  Rings of at most 64 MiB are filled with ordinary
 * stores on the way in, larger ones with non-temporal stores.
 * One stage-out call may mix relay and arena buffers: a rank that keeps training under a new world size
 * relays the part of its new shard it already holds and rests the remainder of its old shard on the
 * host in the same pass.  A non-empty buffer with neither place to go is DR_ERR_INVALID.
 */
typedef struct dr_stage_desc {
    uint32_t struct_size, n_bufs;       /* sizeof(dr_stage_desc); 1..DR_MAX_STAGE_BUFS                */
    void* dev_ptr[DR_MAX_STAGE_BUFS];   /* device buffers, in stream order                            */
    uint64_t bytes[DR_MAX_STAGE_BUFS];
    uint32_t order[DR_MAX_STAGE_BUFS];  /* stage-in priority, a permutation of 0..n_bufs-1            */
    uint64_t budget_bytes;
    uint64_t chunk_bytes;               /* 0: budget / 2 rounded down to a multiple of 4096; but where
                                           the bytes pass through the ring (a relay target, a pageable
                                           arena) at most 4 MiB on the way out and 8 MiB on the way in,
                                           in a ring of at most 64 MiB (the fast geometry, see above)  */
    void* host_arena;
    uint64_t host_arena_bytes;
    dr_chunk_fn callback;
    void* user;
    void* relay_dev[DR_MAX_STAGE_BUFS];
    uint64_t first_chunk;               /* resume: chunks / pieces below this index are skipped       */
    void* wait_event;                   /* cudaEvent_t the first copy waits for INSTEAD of
                                           caller_stream's pending work: the overlap recipe records
                                           it before enqueueing dr_reshard, so that stage-out starts
                                           while the repack runs (both only read).  NULL: none      */
    void* ready_events[DR_MAX_STAGE_BUFS]; /* stage-in: caller's cudaEvent_t recorded on the copy
                                              stream right after buffer i's last copy; NULL = none   */
    uint32_t timeout_ms;                /* bound on every internal wait; 0 = 60 000                   */
    uint32_t flags;                     /* DR_STAGE_HOST_OFFSETS | DR_STAGE_UNORDERED, or 0           */
    uint64_t host_offset[DR_MAX_STAGE_BUFS]; /* with DR_STAGE_HOST_OFFSETS: buffer i rests at
                                           host_arena + host_offset[i] instead of at its position in
                                           the stream; regions must not overlap (arena sinks only)    */
    void* caller_stream;                /* cudaStream_t on which the caller produced (stage-out) or
                                           last used (stage-in, relay targets) the device buffers;
                                           NULL = the legacy default stream.  Unless wait_event or
                                           DR_STAGE_UNORDERED is given, the first copy waits for all
                                           work enqueued on it before the call                        */
    void* done_event;                   /* caller's cudaEvent_t recorded after the call's last copy
                                           (already complete when the call returns), or NULL          */
} dr_stage_desc;

/* Buffer i of a stage call rests at host_arena + host_offset[i].  This is how training state crosses a
 * change of the training world size (Sec. 3.3, old ranks -> new ranks through host memory): every old
 * rank stages its shard out to its place in one flat host image, every new rank stages its own,
 * differently cut, range back in (see dr_shard_range). */
#define DR_STAGE_HOST_OFFSETS 1u
/* The caller has ordered the device buffers itself (a synchronise, or its own events): the call neither
 * records on nor waits for caller_stream. */
#define DR_STAGE_UNORDERED 2u

typedef struct dr_stage_stats {
    uint64_t bytes;                    /* bytes moved by this call                                    */
    uint64_t chunks_done;              /* chunks (stage-out) / pieces (stage-in) complete, counted
                                          from 0: on failure, resume with first_chunk = chunks_done  */
    uint64_t n_chunks;                 /* total for the whole stream                                  */
    double elapsed_ms;
    double link_gbs;                   /* bytes / elapsed, 1e9 bytes per second                       */
    uint64_t pinned_high_water_bytes;  /* pinned ring bytes held (0 when a pinned arena is used)      */
    double ready_ms[DR_MAX_STAGE_BUFS];/* stage-in: time from call start until buffer i was resident  */
} dr_stage_stats;

/*
 * dr_stage_out -- device -> host in bounded chunks (Sec. 3.3: the states are partitioned into
 * chunks and streamed through host-memory buffers, store and reload pipelined chunk by chunk).
 * Blocking pump on the calling thread; copies run on the plan's side stream.  Overlap recipe: record
 * an event on the caller's stream once the state buffers are final, enqueue dr_reshard, then call
 * dr_stage_out with wait_event = that event: the copies start while the repack runs (both only read
 * the master buffer).  Without wait_event the first copy waits for all of caller_stream's pending
 * work, the repack included.  On return every delivered chunk is complete and byte-exact.  Errors: DR_ERR_INVALID, DR_ERR_BUDGET, DR_ERR_SIZE (arena too small),
 * DR_ERR_NOMEM (pinned ring), DR_ERR_SINK, DR_ERR_TIMEOUT, DR_ERR_CUDA, DR_ERR_STATE.
 * Stage calls on one plan share its ring and are serialised inside the library (a second thread's call
 * waits for the first to return).
 */
int dr_stage_out(dr_plan* plan, const dr_stage_desc* desc, dr_stage_stats* stats);

/*
 * dr_stage_in -- host -> device, buffers in desc->order so that the weights are resident first and
 * the optimizer state follows (Sec. 3.3: only the weights are loaded during the transition, the
 * optimizer states are deferred to the first step on the new topology).  stats->ready_ms[i] and
 * ready_events[i] tell when buffer i became usable.  The first copy is ordered after caller_stream's
 * pending work (a zero-fill or an allocation reuse of the target buffers must not land after it).
 * Same pump, errors and threading as above.
 */
int dr_stage_in(dr_plan* plan, const dr_stage_desc* desc, dr_stage_stats* stats);

/*
 * Deferred form of the two calls above (Sec. 3.3: only the weights are needed at the transition; the
 * optimizer states are reloaded off the critical path, while the first step on the new topology is
 * being prepared).  dr_stage_begin checks the descriptor, fixes the ordering point (everything enqueued
 * on desc->caller_stream up to this call, or desc->wait_event) and starts the same pump on a thread the
 * library owns; it returns at once.  The caller goes on (typically: runs dr_reshard_inverse, waits for the weights with
 * dr_stage_wait_buffer, starts the step) and later collects the result:
 *   dr_stage_wait_buffer : (stage-in) blocks the calling thread, at most timeout_ms (0 = 60 s), until
 *                   buffer i is resident: its last copy has completed, so work enqueued afterwards on any
 *                   stream may use it.  This is the way to wait for the weights here: ready_events[i] is
 *                   recorded by the library's thread when the buffer's last copy is enqueued, and a
 *                   cudaStreamWaitEvent on an event that has not been recorded yet does not wait at all.
 *                   DR_ERR_TIMEOUT; the job's own error if the pump ended without the buffer.
 *   dr_stage_poll : *done = 1 once the pump has returned (never blocks)
 *   dr_stage_end  : waits for the pump, fills stats, returns the status dr_stage_out / dr_stage_in
 *                   would have returned (with its message in dr_last_error) and frees the job
 * direction: DR_STAGE_DIR_OUT or DR_STAGE_DIR_IN.  The descriptor is copied; the buffers, the arena, the
 * events and the callback it names must stay valid until dr_stage_end.  A callback runs on the library's
 * thread.  Every job must be ended before its plan is destroyed; jobs on one plan run one after the
 * other.  Errors of dr_stage_begin: DR_ERR_INVALID, DR_ERR_BUDGET, DR_ERR_SIZE, DR_ERR_STATE (found
 * before anything is started), DR_ERR_NOMEM, DR_ERR_CUDA.
 */
typedef struct dr_stage_job dr_stage_job;
enum { DR_STAGE_DIR_OUT = 0, DR_STAGE_DIR_IN = 1 };
int dr_stage_begin(dr_plan* plan, const dr_stage_desc* desc, int direction, dr_stage_job** job);
int dr_stage_wait_buffer(dr_stage_job* job, uint32_t buffer, uint32_t timeout_ms);
int dr_stage_poll(const dr_stage_job* job, int* done);
int dr_stage_end(dr_stage_job* job, dr_stage_stats* stats);

/*
 * Streamed repack: Training -> Rollout for a GPU that does not hold the fp32 master.  The flat source
 * rests in pinned host memory (where dr_stage_out left it); it is copied to the device chunk by chunk
 * into a caller-provided window of a few chunks, each chunk is repacked as soon as it has arrived, and
 * (optionally) every range of the rollout arena is copied back to pinned host memory as soon as no later
 * chunk can write into it.  Host-to-device copies, the repack kernels and device-to-host copies run on
 * three streams and overlap, so the whole switch takes about as long as the larger of the two copy
 * directions; the device never holds more than the window of fp32 state (the bounded staging of Sec. 3.3
 * applied to the device side, and Sec. 3.3's overlap of operations that do not depend on one another).
 */
typedef struct dr_stream_desc {
    uint32_t struct_size, flags;  /* sizeof(dr_stream_desc); 0 or DR_STREAM_UNORDERED                  */
    const void* host_src;         /* pinned host: the plan's source buffer (dr_plan_query: src_bytes)  */
    uint64_t host_src_bytes;
    void* dst_dev;                /* device: the rollout arena                                         */
    uint64_t dst_bytes;
    void* host_dst;               /* pinned host copy of the arena, or NULL                            */
    uint64_t host_dst_bytes;
    void* window_dev;             /* device scratch the caller owns: slots = floor(window / chunk) >= 2 */
    uint64_t window_bytes;
    uint64_t chunk_bytes;         /* multiple of 32; 0: window_bytes / 2 rounded down to 4096, at most
                                     32 MiB (at most 16 chunks of the window are in use at a time)      */
    uint32_t timeout_ms;          /* bound on the final wait; 0 = 60 000                               */
    uint32_t pad;
    void* caller_stream;          /* cudaStream_t on which the caller last touched dst_dev / window_dev
                                     (e.g. filled or zeroed them); NULL = the legacy default stream.  All
                                     work enqueued on it before the call completes before the first copy
                                     or kernel of the call, unless wait_event or DR_STREAM_UNORDERED      */
    void* wait_event;             /* cudaEvent_t to wait for instead of caller_stream's pending work      */
    void* done_event;             /* caller's cudaEvent_t recorded after the last kernel and copy, or NULL */
} dr_stream_desc;

/* The caller has ordered dst_dev and window_dev itself: no record on / wait for caller_stream. */
#define DR_STREAM_UNORDERED 1u

typedef struct dr_stream_stats {
    uint64_t h2d_bytes, d2h_bytes, n_chunks, kernels;
    double elapsed_ms;            /* first enqueue to everything complete                              */
} dr_stream_stats;

/*
 * dr_reshard_stream -- the result in dst_dev (and host_dst) is exactly dr_reshard's on the same source.
 * Blocking: returns when every copy and kernel has completed (bounded poll, DR_ERR_TIMEOUT).  The first
 * call with a given chunk size compiles and uploads one small segment table per chunk (device memory
 * owned by the plan, re-used by later calls).  On a timeout or an enqueue error the call still waits
 * (bounded, a generous fixed limit) for what it had already enqueued, so that nothing of it is in flight
 * on return.  Errors: DR_ERR_INVALID (bad descriptor; chunk_bytes not a multiple of 32), DR_ERR_SIZE (a
 * buffer too small), DR_ERR_ALIGN (pointers not 32-byte aligned), DR_ERR_BUDGET (window below two chunks),
 * DR_ERR_STATE (host-only plan), DR_ERR_NOMEM, DR_ERR_CUDA, DR_ERR_TIMEOUT.  Calls on one plan must not
 * overlap.
 */
int dr_reshard_stream(dr_plan* plan, const dr_stream_desc* desc, dr_stream_stats* stats);

/*
 * dr_shard_range -- the flat elements [*begin, *end) that rank `rank` of `world` really holds
 * (S = ceil(flat_elems / world) per rank; the last ranks' padding past flat_elems is excluded, so
 * *end - *begin can be smaller than S, or zero).  With it a caller lays out a re-shard across a changed
 * world size (Sec. 3.3: e.g. 6 training GPUs -> 4): the old rank stages out [begin, end) of its shard
 * to host_offset = 4 * begin of a flat host image, the new rank stages in its own range from there, and
 * the part of the new range the GPU already holds can go through a relay sink without touching the
 * image.  Host arithmetic only.  DR_ERR_INVALID for world == 0, rank >= world or NULL outputs.
 */
int dr_shard_range(uint64_t flat_elems, uint32_t world, uint32_t rank, uint64_t* begin, uint64_t* end,
                   uint64_t* shard_elems);

/*
 * Hysteresis-guided reconfiguration (Sec. 3.4; host only, no CUDA).  The controller only decides WHEN to
 * move between pre-specified topologies, listed from most-Training to most-Rollout (e.g. 6:2, 5:3, 4:4).
 * Per step: imbalance = (t_rollout - t_train) / max(t_rollout, t_train).  A step signals "towards
 * Rollout" if imbalance > enter_threshold, "towards Training" if < -enter_threshold, is quiet if
 * |imbalance| < exit_threshold, and otherwise lies in the hysteresis band (the streak of signals neither
 * grows nor resets).  A move by one position is decided when `consecutive` signals of one direction have
 * arrived in a row, the topology has been held for dwell_steps, the previous move is cooldown_steps ago
 * (Sec. 5 Exp#3: more than 10 steps, above the ~11-step break-even) and the neighbour exists.
 */
typedef struct dr_ctl_config {
    uint32_t struct_size, n_topologies, initial;
    uint32_t consecutive, dwell_steps, cooldown_steps;
    double enter_threshold, exit_threshold; /* 0 <= exit <= enter, enter > 0 */
} dr_ctl_config;
typedef struct dr_ctl dr_ctl;

int dr_ctl_create(const dr_ctl_config* cfg, dr_ctl** out);                /* DR_ERR_INVALID, DR_ERR_NOMEM */
/* Feed one step.  *move = -1 / 0 / +1, *topology = index after the move.  DR_ERR_INVALID on NaN / negative times. */
int dr_ctl_observe(dr_ctl* ctl, double t_rollout, double t_train, int32_t* move, uint32_t* topology);
/* Sustained steps after which one resize has paid for itself: cost / (step_before - step_after) (Exp#3);
 * infinity when the step did not get faster. */
int dr_ctl_break_even(double resize_cost_s, double step_before_s, double step_after_s, double* steps);
int dr_ctl_destroy(dr_ctl* ctl);

/*
 * dr_probe_stream -- measurement aid (the paper has no counterpart): a trivial contiguous streaming
 * kernel in the repack kernel's launch shape, so that a benchmark can measure, in the same run as the
 * repack, what this GPU sustains for the repack's read : write mix.  n_bytes counts the wider side and
 * must be a multiple of 49 152 (one CTA's tile); both buffers 32-byte aligned.
 *   DR_PROBE_READ   reads n_bytes of a_dev                       (b_dev unused, may be NULL)
 *   DR_PROBE_WRITE  writes n_bytes to b_dev                      (a_dev unused, may be NULL)
 *   DR_PROBE_COPY   copies n_bytes a_dev -> b_dev                (1 : 1)
 *   DR_PROBE_NARROW reads n_bytes of fp32, writes n_bytes / 2 of bf16 (2 : 1, the forward repack's mix)
 *   DR_PROBE_WIDEN  reads n_bytes / 2 of bf16, writes n_bytes of fp32 (1 : 2, the inverse map's mix)
 *   DR_PROBE_NARROW4 reads n_bytes, writes n_bytes / 4                (4 : 1, the fp8 forward's mix)
 *   DR_PROBE_WIDEN4  reads n_bytes / 4, writes n_bytes                (1 : 4, the fp8 inverse's mix)
 * Asynchronous on cuda_stream.  Errors: DR_ERR_INVALID, DR_ERR_ALIGN, DR_ERR_UNSUPPORTED, DR_ERR_CUDA.
 */
enum { DR_PROBE_READ = 0, DR_PROBE_WRITE = 1, DR_PROBE_COPY = 2, DR_PROBE_NARROW = 3, DR_PROBE_WIDEN = 4,
       DR_PROBE_NARROW4 = 5, DR_PROBE_WIDEN4 = 6 };
int dr_probe_stream(uint32_t mode, const void* a_dev, void* b_dev, uint64_t n_bytes, void* cuda_stream);

/*
 * dr_host_copy -- measurement aid (the paper has no counterpart): the multi-threaded host copy that the
 * staging engine uses between its pinned ring and a pageable arena (worker threads taking 1 MiB tasks,
 * non-temporal stores), run on its own, so that a benchmark can state what the host's cores sustain
 * without the link (the CPU baseline of staging through pageable memory).  threads = 0 takes the
 * engine's own count (see dr_stage_desc).  Blocking.  DR_ERR_INVALID on NULL.
 */
int dr_host_copy(void* dst_host, const void* src_host, uint64_t n_bytes, uint32_t threads);

/*
 * dr_diag_bulk_wait_failures -- diagnostic (the paper has no counterpart).  The repack kernels move whole
 * contiguous tiles with the TMA unit's bulk copies and wait for them on an mbarrier with an iteration
 * limit; a wait that ran out makes the tile fall back to the register path (same result) and counts
 * here.  *count = such events on the current device since the library was loaded; expected 0.
 * Synchronous (reads a device counter).  DR_ERR_INVALID, DR_ERR_CUDA.
 */
int dr_diag_bulk_wait_failures(uint64_t* count);

/*
 * dr_diag_bulk_starve -- test hook (the paper has no counterpart).  While `on` is non-zero, every tile of the
 * bulk-copy kernel is told to expect 16 bytes more than its copies deliver on the current device, so its
 * bounded wait (about 50 ms) has to run out and the tile is redone by the register path: the way to
 * exercise that path and the counter above without faulting or hanging anything.  The result of
 * dr_reshard stays correct; it is only slow.  Switch it off again with on = 0.  Synchronous.
 */
int dr_diag_bulk_starve(int on);

/* Synchronises the plan's own streams, frees its ring, table and streams.  NULL is accepted. */
int dr_plan_destroy(dr_plan* plan);

const char* dr_strerror(int status);
const char* dr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* DYNARESIZE_H */
