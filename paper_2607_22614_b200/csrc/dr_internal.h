// Internal declarations shared by the planner, the kernels and the staging engine.
#pragma once
#include <cstdint>
#include <cstdio>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "dynaresize.h"

namespace dr {

// A work unit is 8 consecutive elements of one row (32 B of fp32, 16 B of bf16); a tile is
// kTileUnits consecutive units of one segment.  One CTA iteration processes one tile.
#ifndef DR_TILE_UNITS
#define DR_TILE_UNITS 1536
#endif
constexpr uint32_t kUnitElems = 8;
constexpr uint32_t kTileUnits = DR_TILE_UNITS;
// Contiguous runs are cut so that a segment's unit count fits 32 bits with room to spare.
constexpr uint64_t kMaxSegElems = 1ull << 31;
// The tile -> segment hint table has at most this many entries (256 KiB).
constexpr uint64_t kMaxHints = 65536;

enum SegFlags : uint32_t {
    kSegVec32 = 1u,      // flat-side addresses 32-byte aligned: 256-bit accesses allowed
    kSegVec16 = 2u,      // flat-side addresses 16-byte aligned: 128-bit accesses
    kSegContiguous = 4u  // rows == 1: no row/column split needed
};

// Device segment table entry (48 bytes).
struct DevSeg {
    uint64_t dst_off;        // bytes from the arena base
    uint64_t src_off;        // elements from the flat buffer base
    uint64_t tile0;          // index of this segment's first tile
    uint32_t n_units;        // rows * units_per_row
    uint32_t units_per_row;  // ceil(row_len / 8)
    uint32_t row_len;        // elements
    uint32_t src_stride;     // elements
    uint32_t dst_stride;     // elements
    uint32_t flags;
};
static_assert(sizeof(DevSeg) == 48, "DevSeg layout");

// fp8 block quantisation: one entry per quantised rollout tensor, one per row-block source part.
struct QPart {
    uint64_t src_off;   // flat element offset of the part's first row, at the tensor's first column
    uint32_t dst_row0;  // first rollout row the part fills
    uint32_t rows;
    uint32_t src_stride;  // elements between source rows
    uint32_t pad;
};
static_assert(sizeof(QPart) == 24, "QPart layout");
struct QTensor {
    uint64_t payload_off, scale_off;  // arena bytes
    uint64_t block0;                  // index of the tensor's first block
    uint32_t rows, cols, nbc;         // nbc = column blocks
    uint32_t part0, n_parts;
    uint32_t aligned;                 // 1: every source row start and the column count allow 256-bit loads
};
static_assert(sizeof(QTensor) == 48, "QTensor layout");

struct HostSeg {
    uint64_t dst_off, src_off, rows, row_len, src_stride, dst_stride;
    uint32_t flags, tensor;
    uint32_t group = 0;  // 0: embed, 1..L: layers, L+1: final norm and lm_head
};

// A group of rollout tensors that can be repacked on its own (tiles [tile_lo, tile_hi) of the plan).
struct Group {
    uint64_t tile_lo = 0, tile_hi = 0, elems = 0;
    uint64_t qblock_lo = 0, qblock_hi = 0, qelems = 0;  // fp8 plans: the group's quantisation blocks
    uint32_t first_tensor = 0, n_tensors = 0;
};

struct Tensor {
    std::string name;
    uint64_t arena_off = 0, rows = 0, cols = 0;
    int64_t alias_of = -1;
    uint32_t group = 0;
    uint32_t es = 2;         // payload bytes per element
    bool quant = false;
    uint64_t scale_off = 0;  // quantised tensors
};

// Everything a launch needs besides the buffers.
struct Tables {
    std::vector<DevSeg> segs;
    std::vector<uint32_t> hints;
    uint32_t hint_shift = 0;
    uint64_t n_tiles = 0, elems = 0;
};

struct Ring;    // pinned staging ring + worker pool (staging.cu)
struct Stream;  // per-chunk tables of a streamed repack (stream.cu)

}  // namespace dr

struct dr_plan {
    dr_model_spec spec{};
    dr_src_layout src{};
    dr_dst_layout dst{};
    uint32_t tp = 1, tp_rank = 0;
    uint32_t elem_size = 2;  // rollout element size in bytes
    dr_plan_info info{};
    std::vector<dr::Tensor> tensors;
    std::vector<dr::HostSeg> segs;
    std::vector<dr::DevSeg> dev_segs;  // host copy of the device table
    std::vector<dr::Group> groups;
    // hints[i] = segment holding tile i << hint_shift: a tile finds its segment with one load plus a short walk
    std::vector<uint32_t> hints;
    uint32_t hint_shift = 0;
    // fp8 plans: quantised tensors, their parts, and a block -> tensor hint table
    bool fp8 = false;
    std::vector<dr::QTensor> qtensors;
    std::vector<dr::QPart> qparts;
    std::vector<uint32_t> qhints;
    uint32_t qhint_shift = 0;
    // device side (absent on a host-only plan)
    bool host_only = true;
    int device = -1;
    dr::DevSeg* d_segs = nullptr;
    uint32_t* d_hints = nullptr;
    dr::QTensor* d_qtensors = nullptr;
    dr::QPart* d_qparts = nullptr;
    uint32_t* d_qhints = nullptr;
    int grid = 0;
    // forward launches take the TMA bulk-copy kernel (see reshard.cu): set when next to none of the plan's elements
    // sit in strided (column-sliced) segments, whose short per-row copies are slower that way than from registers
    bool bulk_forward = false;
    // staging
    std::mutex stage_mu;
    dr::Ring* ring = nullptr;
    dr::Stream* stream = nullptr;
};

// Run a CUDA runtime call inside a function (or lambda) that returns a dr_status; on failure record the
// message, clear the (non-sticky) error so that later launches do not see it, and return.
#define DR_CUDA(call)                                                             \
    do {                                                                          \
        cudaError_t e_ = (call);                                                  \
        if (e_ != cudaSuccess) {                                                  \
            cudaGetLastError();                                                   \
            dr::set_error("%s: %s", #call, cudaGetErrorString(e_));               \
            return e_ == cudaErrorMemoryAllocation ? DR_ERR_NOMEM : DR_ERR_CUDA;  \
        }                                                                         \
    } while (0)

namespace dr {

void set_error(const char* fmt, ...);
int compile_plan(dr_plan* p);  // planner.cpp: fills tensors, segs, dev_segs, info
// Tiles [tile_lo, min(tile_hi, all)) of the plan.
int launch_reshard(const dr_plan* p, bool inverse, const void* flat, void* arena_or_flat_out, const void* arena_in,
                   void* stream, uint64_t tile_lo = 0, uint64_t tile_hi = ~0ull);
// Forward repack into several arenas at once (the fused exchange).
int launch_push(const dr_plan* p, const void* flat, void* const* arenas, uint32_t n_dst, void* stream);
std::vector<dr_range> plan_ranges(const dr_plan* p);  // planner.cpp: coalesced arena byte ranges the plan writes
int ensure_bulk_smem(int device);          // once per device: lets the repack kernels ask for their tile buffers
int bulk_starve(int on);                   // test hook: makes the bulk tiles' bounded waits run out
int bulk_wait_failures(uint64_t* out);     // bounded mbarrier waits that ran out since the library was loaded (expected: 0)
int choose_grid(int device, uint32_t elem_size);  // resident CTAs of the reshard kernel on the whole GPU
// Blocks [block_lo, min(block_hi, all)) of the plan's quantised tensors.
int launch_quant(const dr_plan* p, const void* flat, void* arena, void* stream, uint64_t block_lo = 0,
                 uint64_t block_hi = ~0ull);
int launch_dequant(const dr_plan* p, const void* arena, void* flat, void* stream);
void ring_destroy(Ring* r);
void stream_destroy(Stream* s);
int build_tables(const std::vector<HostSeg>& segs, Tables* out);
std::vector<HostSeg> window_segments(const std::vector<HostSeg>& segs, uint64_t lo, uint64_t hi, uint32_t es);
// Enqueue the forward kernel for an explicit table (used by the streamed repack).
int launch_forward_tables(uint32_t elem_size, const DevSeg* d_segs, uint32_t n_segs, const uint32_t* d_hints,
                          uint32_t hint_shift, uint64_t n_tiles, const void* flat, void* arena, void* stream, bool bulk);

}  // namespace dr
