// Gather / permute / cast kernels for sm_100a.
//
// The transform is pure data movement (4 B read + 2 B written per element, no contraction), so the
// design goal is HBM bandwidth: every thread keeps three 256-bit loads in flight, each warp-level
// access is one fully coalesced 1 KB (load) or 512 B (store) request, the flat buffer and the arena are
// streamed past L1, and a tile finds its segment with one hint load plus a short walk instead of a
// per-element lookup.  One CTA of 512 threads handles one 48 KB tile (three units per thread) and CTAs are
// dispatched in tile order: measured on B200 this keeps the set of DRAM pages in use compact and runs 12 %
// faster (7.1-7.2 vs 6.4 TB/s) than a persistent grid whose CTAs drift apart; the persistent forms remain
// as compile-time options.  With exactly one tile per CTA the body runs once and needs no loop state.
#include <cuda_runtime.h>

#include "dr_internal.h"

namespace dr {
namespace {

// Compile-time tuning knobs (the defaults are the measured best on B200).
#ifndef DR_THREADS
#define DR_THREADS 512
#endif
#ifndef DR_MIN_BLOCKS
#define DR_MIN_BLOCKS 1
#endif
#ifndef DR_BLOCKED
#define DR_BLOCKED false
#endif
#ifndef DR_GRID_MULT
#define DR_GRID_MULT 0  // 0: one CTA per DR_TILES_PER_CTA tiles; k > 0: persistent grid of k x resident CTAs
#endif
#ifndef DR_TILES_PER_CTA
#define DR_TILES_PER_CTA 1
#endif
#ifndef DR_OCC_SMEM
#define DR_OCC_SMEM 0  // bytes of (unused) dynamic shared memory per CTA: caps the CTAs resident on an SM
#endif
// dynamic shared memory a forward launch asks for: the bulk path's tile buffers, or the occupancy knob above
#define DR_DYN_SMEM ((DR_BULK && DR_GRID_MULT == 0 && DR_TILES_PER_CTA == 1) ? (int)kBulkSmemBytes : DR_OCC_SMEM)
#ifndef DR_LD_HINT
#define DR_LD_HINT ".nc.L1::no_allocate"
#endif
#ifndef DR_ST_HINT
#define DR_ST_HINT ".L1::no_allocate"
#endif
#ifndef DR_LD256_HINT
#define DR_LD256_HINT DR_LD_HINT
#endif
#ifndef DR_ST256_HINT
#define DR_ST256_HINT DR_ST_HINT
#endif
#ifndef DR_BULK
#define DR_BULK 1  // forward tiles go through the TMA unit's 1-D bulk copies and shared memory
#endif

constexpr int kThreads = DR_THREADS;
// The default launch gives every CTA exactly one tile: the kernel body then runs once, without loop state.
constexpr bool kOneTile = (DR_GRID_MULT == 0) && (DR_TILES_PER_CTA == 1);
constexpr int kUnroll = kTileUnits / kThreads;  // units per thread per tile
static_assert(kTileUnits % kThreads == 0, "tile must be a whole number of thread sweeps");

// ---- memory access helpers (inline PTX: 256-bit accesses and cache hints) ----------------------
struct V8 {
    uint32_t w[8];
};
struct V4 {
    uint32_t w[4];
};

__device__ __forceinline__ V8 ld256(const void* p)
{
    V8 v;
    asm volatile("ld.global" DR_LD256_HINT ".v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]), "=r"(v.w[5]), "=r"(v.w[6]),
                   "=r"(v.w[7])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ V4 ld128(const void* p)
{
    V4 v;
    asm volatile("ld.global" DR_LD_HINT ".v4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3])
                 : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ld32(const void* p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ uint16_t ld16(const void* p)
{
    uint16_t v;
    asm volatile("ld.global.nc.L1::no_allocate.b16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st256(void* p, const V8& v)
{
    asm volatile("st.global" DR_ST256_HINT ".v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]),
                 "r"(v.w[2]), "r"(v.w[3]), "r"(v.w[4]), "r"(v.w[5]), "r"(v.w[6]), "r"(v.w[7])
                 : "memory");
}
__device__ __forceinline__ void st128(void* p, const V4& v)
{
    asm volatile("st.global" DR_ST_HINT ".v4.b32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.w[0]), "r"(v.w[1]),
                 "r"(v.w[2]), "r"(v.w[3])
                 : "memory");
}
__device__ __forceinline__ void st32(void* p, uint32_t v)
{
    asm volatile("st.global.L1::no_allocate.b32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st16(void* p, uint16_t v)
{
    asm volatile("st.global.L1::no_allocate.b16 [%0], %1;" ::"l"(p), "h"(v) : "memory");
}

// fp32 -> bf16, round to nearest even, in hardware: NaN becomes 0x7FFF, subnormals are rounded (the
// instruction has no flush-to-zero form), overflow goes to infinity.
__device__ __forceinline__ uint32_t cvt_pair(uint32_t lo, uint32_t hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(__uint_as_float(hi)), "f"(__uint_as_float(lo)));
    return d;
}
__device__ __forceinline__ uint16_t cvt_one(uint32_t x)
{
    uint16_t d;
    asm("cvt.rn.bf16.f32 %0, %1;" : "=h"(d) : "f"(__uint_as_float(x)));
    return d;
}
__device__ __forceinline__ V4 narrow(const V8& v)
{
    V4 o;
    o.w[0] = cvt_pair(v.w[0], v.w[1]);
    o.w[1] = cvt_pair(v.w[2], v.w[3]);
    o.w[2] = cvt_pair(v.w[4], v.w[5]);
    o.w[3] = cvt_pair(v.w[6], v.w[7]);
    return o;
}
__device__ __forceinline__ V8 widen(const V4& v)
{
    V8 o;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        o.w[2 * i] = v.w[i] << 16;
        o.w[2 * i + 1] = v.w[i] & 0xFFFF0000u;
    }
    return o;
}

// flat side: fp32 at 16- or 32-byte aligned addresses
__device__ __forceinline__ V8 load_flat(const char* p, bool wide)
{
    if (wide) return ld256(p);
    V4 a = ld128(p), b = ld128(p + 16);
    return V8{{a.w[0], a.w[1], a.w[2], a.w[3], b.w[0], b.w[1], b.w[2], b.w[3]}};
}
__device__ __forceinline__ void store_flat(char* p, const V8& v, bool wide)
{
    if (wide) {
        st256(p, v);
    } else {
        st128(p, V4{{v.w[0], v.w[1], v.w[2], v.w[3]}});
        st128(p + 16, V4{{v.w[4], v.w[5], v.w[6], v.w[7]}});
    }
}

// Last segment whose first tile is <= tile, searching upward from `from`.
__device__ __forceinline__ uint32_t find_segment(const DevSeg* __restrict__ segs, uint32_t n_segs, uint32_t from,
                                                 uint64_t tile)
{
    // the common case is one of the next few entries
    uint32_t s = from;
#pragma unroll 1
    for (int probe = 0; probe < 4; ++probe) {
        if (s + 1 >= n_segs || segs[s + 1].tile0 > tile) return s;
        ++s;
    }
    uint32_t lo = s, hi = n_segs;  // invariant: segs[lo].tile0 <= tile, (hi == n_segs or segs[hi].tile0 > tile)
    while (hi - lo > 1) {
        uint32_t mid = lo + (hi - lo) / 2;
        if (segs[mid].tile0 <= tile) lo = mid; else hi = mid;
    }
    return lo;
}

// Further arenas that receive every element the forward kernel produces (the fused exchange): own memory or
// peers' memory reached by plain stores.  The kernel's `arena` argument is destination 0; these are 1..n.
struct Peers {
    char* a[DR_MAX_PUSH_DST - 1];
    uint32_t n;
};

// ---- forward tiles through the TMA unit -------------------------------------------------------------------------
// A forward tile of a vector-class segment comes in by 1-D bulk asynchronous copies (cp.async.bulk: no tensor map,
// no multicast): global -> shared memory, one copy per source row the tile touches (one in all for a contiguous
// run), completion counted in bytes on an mbarrier.  It leaves through registers: 16 bytes read from shared memory,
// cast, one 64-bit (bf16) or 128-bit (fp32) global store per thread and step, every warp one contiguous request.
// Measured on B200, the 8.19 G-element contiguous plan, per launch: from idle (SM clock 1965 MHz) 6.80-6.87 ms
// against 6.90-6.95 ms for the register kernel; in a long run of launches, with the part at its power limit and the
// SM clock near 1.6 GHz, 6.87-6.88 ms against 6.89 ms.  DR_BULK_STORE=1 keeps the earlier form, which also casts from
// shared to shared memory and stores the tile with one bulk copy: 6.80-6.82 ms from idle, but 7.04-7.2 ms at the
// power limit (it leans on the TMA unit twice per byte and follows the SM clock down), so it is not the default.
// It is used for the forward direction only: for the write-heavy inverse the register path is the faster one, and a
// kernel that reserves the tile buffers leaves the register path too little L1 to keep its loads in flight, so
// the two are not mixed in one launch configuration.
// The wait on the mbarrier is bounded.  If it ever ran out, the tile is redone by the register path (same result)
// after the copies in flight have been given a second bounded wait, and a counter is raised for the host to read.
constexpr uint32_t kTileFlatBytes = kTileUnits * 32;                      // 48 KB of fp32
#ifndef DR_BULK_STORE
#define DR_BULK_STORE 0
#endif
constexpr uint32_t kBulkSmemBytes = DR_BULK_STORE ? kTileFlatBytes + kTileFlatBytes / 2 : kTileFlatBytes;  // (+ 24 KB of bf16)
constexpr uint32_t kBulkMaxRows = 32;                                     // source rows per tile the first warp can issue
__device__ unsigned int g_bulk_wait_gave_up = 0;
// Test hook: when set, every bulk tile expects 16 bytes more than its copies deliver, so its wait has to run out.
__device__ unsigned int g_bulk_starve = 0;

__device__ __forceinline__ uint64_t global_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for the barrier's phase `parity`, at most about 50 ms (and never more than 2^22 polls): a tile's copies take
// microseconds, so a wait that long has failed.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity)
{
    uint32_t done = 0;
    const uint64_t t0 = global_ns();
#pragma unroll 1
    for (uint32_t it = 0; it < (1u << 22) && !done; ++it) {
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done)
                     : "r"(bar), "r"(parity)
                     : "memory");
        if (!done && (it & 63) == 63 && global_ns() - t0 > 50000000ull) break;
    }
    return done != 0;
}

// Units [ub, ub + n) of segment g, flat -> arena(s).  Returns false if the tile has to take the register path.
template <int ES>
__device__ __forceinline__ bool bulk_forward_tile(const DevSeg& g, uint32_t ub, uint32_t n, const char* fbase, char* arena,
                                                  char* smem, uint64_t* bar_ptr)
{
    const bool contiguous = g.flags & kSegContiguous;
    // source pieces: piece 0 is the rest of the first row, the others are whole rows, the last may be cut short
    const uint32_t upr = contiguous ? n : g.units_per_row;
    const uint32_t row0 = contiguous ? 0 : ub / upr, c0 = contiguous ? ub : ub - row0 * upr;
    const uint32_t n0 = contiguous ? n : min(upr - c0, n);
    const uint32_t pieces = 1 + (n - n0 + upr - 1) / upr;
    if (pieces > kBulkMaxRows || (!contiguous && g.dst_stride != g.row_len)) return false;
    char* in = smem;
    char* out = ES == 4 ? smem : smem + kTileFlatBytes;  // layout-only plans store what they loaded
    const uint32_t bar = (uint32_t)__cvta_generic_to_shared(bar_ptr);
    const uint32_t in_s = (uint32_t)__cvta_generic_to_shared(in), out_s = (uint32_t)__cvta_generic_to_shared(out);
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n * 32u + (g_bulk_starve ? 16u : 0u))
                     : "memory");
    }
    if (threadIdx.x < 32) {
        __syncwarp();  // the byte count is expected before the first copy can complete
        if (threadIdx.x < pieces) {
            const uint32_t i = threadIdx.x;
            const uint32_t cnt = i == 0 ? n0 : min(upr, n - n0 - (i - 1) * upr);
            const uint32_t at = i == 0 ? 0 : n0 + (i - 1) * upr;  // units of the tile before this piece
            const char* src = contiguous ? fbase + (uint64_t)ub * 32
                                         : fbase + ((uint64_t)(row0 + i) * g.src_stride + (i == 0 ? c0 * 8 : 0)) * 4;
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             in_s + at * 32),
                         "l"(src), "r"(cnt * 32u), "r"(bar)
                         : "memory");
        }
    }
    __syncthreads();  // the barrier is initialised before anyone polls it
    if (!mbar_wait_bounded(bar, 0)) {
        if (threadIdx.x == 0) atomicAdd(&g_bulk_wait_gave_up, 1u);
        mbar_wait_bounded(bar, 0);  // the copies must not land in the shared memory of a CTA that has moved on
        return false;
    }
#if !DR_BULK_STORE
    {   // out of shared memory through registers: cast, and plain stores (each warp one contiguous 256 or 512 B request)
        char* dst = arena + g.dst_off + (uint64_t)ub * 8 * ES;
#pragma unroll 2
        for (uint32_t q = threadIdx.x; q < n * 2; q += kThreads) {
            const uint4 v = *reinterpret_cast<const uint4*>(in + q * 16);
            if (ES == 2)
                asm volatile("st.global.L1::no_allocate.v2.b32 [%0], {%1,%2};" ::"l"(dst + q * 8), "r"(cvt_pair(v.x, v.y)),
                             "r"(cvt_pair(v.z, v.w))
                             : "memory");
            else
                asm volatile("st.global.L1::no_allocate.v4.b32 [%0], {%1,%2,%3,%4};" ::"l"(dst + q * 16), "r"(v.x), "r"(v.y),
                             "r"(v.z), "r"(v.w)
                             : "memory");
        }
        (void)out_s;
        return true;
    }
#endif
    if (ES == 2) {  // fp32 -> bf16: 16 bytes in, 8 bytes out per step, consecutive threads consecutive quads
#pragma unroll 2
        for (uint32_t q = threadIdx.x; q < n * 2; q += kThreads) {
            const uint4 v = *reinterpret_cast<const uint4*>(in + q * 16);
            *reinterpret_cast<uint2*>(out + q * 8) = make_uint2(cvt_pair(v.x, v.y), cvt_pair(v.z, v.w));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes before the async-proxy read
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        // the rollout side of the tile is dense: it starts ub units into the segment
        const uint64_t off = g.dst_off + (uint64_t)ub * 8 * ES;
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(arena + off), "r"(out_s),
                     "r"(n * 8u * ES)
                     : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // shared memory is read out before the CTA leaves
    }
    return true;
}

// ES: rollout element size (2 = bf16, 4 = fp32).  INV: false = flat -> arena, true = arena -> flat.
// BLOCKED: each CTA takes one contiguous range of tiles; otherwise tiles are dealt round-robin.
// PUSH: forward only; every store is repeated into peers.a[0 .. peers.n).
// BULK: forward only; vector-class tiles go through the TMA unit and shared memory (launched with kBulkSmemBytes).
template <int ES, bool INV, bool BLOCKED, bool PUSH = false, bool BULK = false>
__global__ void __launch_bounds__(kThreads, DR_MIN_BLOCKS)
    reshard_kernel(const DevSeg* __restrict__ segs, uint32_t n_segs, const uint32_t* __restrict__ hints,
                   uint32_t hint_shift, uint64_t tile_begin, uint64_t n_tiles, char* __restrict__ flat,
                   char* __restrict__ arena, int allow256, Peers peers = Peers{})
{
    // this launch covers tiles [tile_begin, n_tiles)
    uint64_t tile, last, step;
    if (BLOCKED) {
        uint64_t per = (n_tiles - tile_begin + gridDim.x - 1) / gridDim.x;
        tile = tile_begin + per * blockIdx.x;
        last = tile + per < n_tiles ? tile + per : n_tiles;
        step = 1;
    } else {
        tile = tile_begin + blockIdx.x;
        last = n_tiles;
        step = gridDim.x;
    }
    if (tile >= last) return;

    uint32_t si = find_segment(segs, n_segs, hints[tile >> hint_shift], tile);
    DevSeg g = segs[si];
    uint64_t seg_end = si + 1 < n_segs ? segs[si + 1].tile0 : n_tiles;

    for (;;) {
        if (!kOneTile && tile >= seg_end) {
            uint32_t h = hints[tile >> hint_shift];
            si = find_segment(segs, n_segs, h > si ? h : si, tile);
            g = segs[si];
            seg_end = si + 1 < n_segs ? segs[si + 1].tile0 : n_tiles;
        }
        const uint32_t u0 = (uint32_t)(tile - g.tile0) * kTileUnits + threadIdx.x;
        const char* fbase = flat + g.src_off * 4;
        char* abase = arena + g.dst_off;
        const bool contiguous = g.flags & kSegContiguous;

#if DR_BULK
        if (BULK && kOneTile && !INV && !PUSH && (g.flags & (kSegVec32 | kSegVec16))) {  // a forward tile whose rows are 16-byte aligned
            extern __shared__ __align__(128) char bulk_smem[];
            __shared__ __align__(8) uint64_t bulk_bar;
            const uint32_t ub = (uint32_t)(tile - g.tile0) * kTileUnits;
            const uint32_t n = min(kTileUnits, g.n_units - ub);
            if (bulk_forward_tile<ES>(g, ub, n, fbase, arena, bulk_smem, &bulk_bar)) return;
        }
#endif

        if (g.flags & (kSegVec32 | kSegVec16)) {
            const bool wide = (g.flags & kSegVec32) && allow256;
            uint64_t fo[kUnroll], ao[kUnroll];
            bool ok[kUnroll];
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                uint32_t u = u0 + j * kThreads;
                ok[j] = u < g.n_units;
                if (contiguous) {
                    fo[j] = (uint64_t)u * 8;
                    ao[j] = (uint64_t)u * 8;
                } else {
                    uint32_t row = u / g.units_per_row;
                    uint32_t col = (u - row * g.units_per_row) * 8;
                    fo[j] = (uint64_t)row * g.src_stride + col;
                    ao[j] = (uint64_t)row * g.dst_stride + col;
                }
            }
            if (!INV) {
                V8 v[kUnroll];
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (ok[j]) v[j] = load_flat(fbase + fo[j] * 4, wide);
#pragma unroll
                for (int j = 0; j < kUnroll; ++j) {
                    if (!ok[j]) continue;
                    if (ES == 2) {
                        const V4 o = narrow(v[j]);
                        st128(abase + ao[j] * 2, o);
                        if (PUSH) {  // fully unrolled: a run-time index would force the pointer array into local memory
#pragma unroll
                            for (uint32_t q = 0; q < DR_MAX_PUSH_DST - 1; ++q)
                                if (q < peers.n) st128(peers.a[q] + g.dst_off + ao[j] * 2, o);
                        }
                    } else {
                        store_flat(abase + ao[j] * 4, v[j], allow256);
                        if (PUSH) {
#pragma unroll
                            for (uint32_t q = 0; q < DR_MAX_PUSH_DST - 1; ++q)
                                if (q < peers.n) store_flat(peers.a[q] + g.dst_off + ao[j] * 4, v[j], allow256);
                        }
                    }
                }
            } else if (ES == 2) {
                V4 v[kUnroll];
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (ok[j]) v[j] = ld128(abase + ao[j] * 2);
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (ok[j]) store_flat((char*)fbase + fo[j] * 4, widen(v[j]), wide);
            } else {
                V8 v[kUnroll];
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (ok[j]) v[j] = load_flat(abase + ao[j] * 4, allow256);
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (ok[j]) store_flat((char*)fbase + fo[j] * 4, v[j], wide);
            }
        } else {
            // Scalar path for runs that start or end off the vector grid (odd shapes, shard cuts):
            // consecutive threads take consecutive elements of the tile, so accesses stay coalesced.
            const uint64_t e0 = (uint64_t)(tile - g.tile0) * kTileUnits * 8;
#pragma unroll 1
            for (uint32_t k = threadIdx.x; k < kTileUnits * 8; k += kThreads) {
                uint64_t e = e0 + k;  // element index in the segment's padded unit space
                uint64_t row, col;
                if (contiguous) {
                    row = 0;
                    col = e;
                } else {
                    uint64_t per_row = (uint64_t)g.units_per_row * 8;
                    row = e / per_row;
                    col = e - row * per_row;
                }
                if (col >= g.row_len || row * g.units_per_row >= g.n_units) continue;
                const char* fp = fbase + (row * g.src_stride + col) * 4;
                char* ap = abase + (row * g.dst_stride + col) * ES;
                if (!INV) {
                    uint32_t x = ld32(fp);
                    if (ES == 2) st16(ap, cvt_one(x)); else st32(ap, x);
                    if (PUSH) {
                        const uint64_t off = g.dst_off + (row * g.dst_stride + col) * ES;
#pragma unroll
                        for (uint32_t q = 0; q < DR_MAX_PUSH_DST - 1; ++q) {
                            if (q >= peers.n) continue;
                            if (ES == 2) st16(peers.a[q] + off, cvt_one(x)); else st32(peers.a[q] + off, x);
                        }
                    }
                } else {
                    uint32_t x = ES == 2 ? (uint32_t)ld16(ap) << 16 : ld32(ap);
                    st32((char*)fp, x);
                }
            }
        }
        if (kOneTile) break;
        tile += step;
        if (tile >= last) break;
    }
}

}  // namespace

// The bulk path's tile buffers exceed the default 48 KB of dynamic shared memory: every instantiation that is launched
// with them is told so once per device.
int ensure_bulk_smem(int device)
{
    if (DR_DYN_SMEM < 40 * 1024) return DR_OK;  // static shared memory counts against the 48 KB default too
    static std::mutex mu;
    static bool done[64] = {false};
    std::lock_guard<std::mutex> lock(mu);
    if (device < 0 || device >= 64) {
        set_error("device index out of range");
        return DR_ERR_CUDA;
    }
    if (done[device]) return DR_OK;
    DR_CUDA(cudaFuncSetAttribute(reshard_kernel<2, false, DR_BLOCKED, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DR_DYN_SMEM));
    DR_CUDA(cudaFuncSetAttribute(reshard_kernel<4, false, DR_BLOCKED, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DR_DYN_SMEM));
    done[device] = true;
    return DR_OK;
}

int bulk_starve(int on)
{
    const unsigned int v = on ? 1u : 0u;
    DR_CUDA(cudaMemcpyToSymbol(g_bulk_starve, &v, sizeof v));
    return DR_OK;
}

int bulk_wait_failures(uint64_t* out)
{
    unsigned int v = 0;
    DR_CUDA(cudaMemcpyFromSymbol(&v, g_bulk_wait_gave_up, sizeof v));
    *out = v;
    return DR_OK;
}

int choose_grid(int device, uint32_t elem_size)
{
    int sms = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) return 0;
    cudaError_t e = elem_size == 2
        ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reshard_kernel<2, false, DR_BLOCKED>, kThreads, DR_OCC_SMEM)
        : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reshard_kernel<4, false, DR_BLOCKED>, kThreads, DR_OCC_SMEM);
    if (e != cudaSuccess || per_sm <= 0) return 0;
    return DR_GRID_MULT ? sms * per_sm * DR_GRID_MULT : 0x7FFFFFFF;
}

int launch_reshard(const dr_plan* p, bool inverse, const void* flat, void* arena_or_flat_out, const void* arena_in,
                   void* stream, uint64_t tile_lo, uint64_t tile_hi)
{
    // forward: flat = source, arena_or_flat_out = arena.  inverse: arena_in = source, arena_or_flat_out = flat.
    char* f = inverse ? (char*)arena_or_flat_out : (char*)flat;
    char* a = inverse ? (char*)arena_in : (char*)arena_or_flat_out;
    if (tile_hi > p->info.n_tiles) tile_hi = p->info.n_tiles;
    if (tile_lo >= tile_hi) return DR_OK;
    const uint64_t n = tile_hi - tile_lo;
    const int allow256 = (((uintptr_t)f | (uintptr_t)a) & 31) == 0;
    uint64_t want = DR_GRID_MULT ? (uint64_t)p->grid : (n + DR_TILES_PER_CTA - 1) / DR_TILES_PER_CTA;
    uint64_t g64 = n < want ? n : want;
    if (g64 > 0x7FFFFFFFull) {
        set_error("%llu tiles exceed the largest grid", (unsigned long long)g64);
        return DR_ERR_UNSUPPORTED;
    }
    dim3 grid((unsigned)g64), block(kThreads);
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t n_segs = (uint32_t)p->dev_segs.size();
#define DR_LAUNCH(ES, INV, BULK)                                                                                       \
    reshard_kernel<ES, INV, DR_BLOCKED, false, BULK><<<grid, block, (BULK) ? DR_DYN_SMEM : DR_OCC_SMEM, s>>>(          \
        p->d_segs, n_segs, p->d_hints, p->hint_shift, tile_lo, tile_hi, f, a, allow256)
    const bool bulk = DR_BULK && !inverse && p->bulk_forward;
    if (p->elem_size == 2) {
        if (inverse) DR_LAUNCH(2, true, false); else if (bulk) DR_LAUNCH(2, false, true); else DR_LAUNCH(2, false, false);
    } else {
        if (inverse) DR_LAUNCH(4, true, false); else if (bulk) DR_LAUNCH(4, false, true); else DR_LAUNCH(4, false, false);
    }
#undef DR_LAUNCH
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("reshard kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}

int launch_push(const dr_plan* p, const void* flat, void* const* arenas, uint32_t n_dst, void* stream)
{
    const uint64_t n = p->info.n_tiles;
    if (n == 0) return DR_OK;
    if (DR_GRID_MULT || DR_TILES_PER_CTA != 1) {
        set_error("the fused exchange is built for the one-tile-per-CTA launch only");
        return DR_ERR_UNSUPPORTED;
    }
    if (n > 0x7FFFFFFFull) {
        set_error("%llu tiles exceed the largest grid", (unsigned long long)n);
        return DR_ERR_UNSUPPORTED;
    }
    Peers peers{};
    uintptr_t all = (uintptr_t)flat;
    for (uint32_t i = 0; i < n_dst; ++i) {
        all |= (uintptr_t)arenas[i];
        if (i) peers.a[i - 1] = (char*)arenas[i];
    }
    peers.n = n_dst - 1;
    const int allow256 = (all & 31) == 0;  // one flag for all destinations
    dim3 grid((unsigned)n), block(kThreads);
    cudaStream_t s = (cudaStream_t)stream;
    const uint32_t n_segs = (uint32_t)p->dev_segs.size();
    // the register kernel: with several destinations the stream is write-heavy, where the bulk path does not pay
    if (p->elem_size == 2)
        reshard_kernel<2, false, DR_BLOCKED, true><<<grid, block, DR_OCC_SMEM, s>>>(
            p->d_segs, n_segs, p->d_hints, p->hint_shift, 0, n, (char*)flat, (char*)arenas[0], allow256, peers);
    else
        reshard_kernel<4, false, DR_BLOCKED, true><<<grid, block, DR_OCC_SMEM, s>>>(
            p->d_segs, n_segs, p->d_hints, p->hint_shift, 0, n, (char*)flat, (char*)arenas[0], allow256, peers);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("push kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}

int launch_forward_tables(uint32_t elem_size, const DevSeg* d_segs, uint32_t n_segs, const uint32_t* d_hints,
                          uint32_t hint_shift, uint64_t n_tiles, const void* flat, void* arena, void* stream, bool bulk)
{
    if (n_tiles == 0) return DR_OK;
    char* f = (char*)flat;
    char* a = (char*)arena;
    const int allow256 = (((uintptr_t)f | (uintptr_t)a) & 31) == 0;
    const uint64_t want = (n_tiles + DR_TILES_PER_CTA - 1) / DR_TILES_PER_CTA;
    if (want > 0x7FFFFFFFull) {
        set_error("%llu tiles exceed the largest grid", (unsigned long long)want);
        return DR_ERR_UNSUPPORTED;
    }
    dim3 grid((unsigned)want), block(kThreads);
    cudaStream_t s = (cudaStream_t)stream;
#define DR_LAUNCH_T(ES, BULK)                                                                                   \
    reshard_kernel<ES, false, DR_BLOCKED, false, BULK><<<grid, block, (BULK) ? DR_DYN_SMEM : DR_OCC_SMEM, s>>>(    \
        d_segs, n_segs, d_hints, hint_shift, 0, n_tiles, f, a, allow256)
    bulk = bulk && DR_BULK;
    if (elem_size == 2) {
        if (bulk) DR_LAUNCH_T(2, true); else DR_LAUNCH_T(2, false);
    } else {
        if (bulk) DR_LAUNCH_T(4, true); else DR_LAUNCH_T(4, false);
    }
#undef DR_LAUNCH_T
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("reshard kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}

}  // namespace dr

// ------------------------------------------------------------------------------------------------
// Allocation-free forward repack.
//
// The ordinary path keeps the segment table in memory that dr_plan_create obtains with cudaMalloc.
// Some callers must not allocate on the device at the moment of a role switch: a worker whose
// framework has handed the whole GPU to its own caching pool (a fresh cudaMalloc then fails or eats
// the head-room the incoming state needs), and a switch that is overlapping staging copies with the
// repack (cudaMalloc and cudaFree synchronise the device and would stall those copies).  For them the
// table lives in the fixed array below, which every GPU that loads this library holds until exit.
// ------------------------------------------------------------------------------------------------
namespace dr {
namespace {

constexpr uint32_t kStaticMaxSegs = 16384;  // 768 KiB + 256 KiB of hints = 1 MiB; the largest benchmark plan needs 12 482
constexpr uint32_t kStaticSegBytes = kStaticMaxSegs * sizeof(DevSeg);
// segment entries first, then the tile -> segment hint table (at most kMaxHints words)
static __device__ __align__(256) unsigned char g_static_segs[kStaticSegBytes + kMaxHints * sizeof(uint32_t)];

constexpr int kMaxDevices = 64;
struct StaticSlot {
    DevSeg* table = nullptr;  // device address of g_static_segs on that device
    int grid[2] = {0, 0};     // persistent grid for bf16 / fp32 rollout plans
};
StaticSlot g_slots[kMaxDevices];
std::mutex g_slots_mu;

// Once per device, with that device current: the array's name is only a host-side handle, the address
// the kernel needs comes from the runtime.
int static_setup(int device, StaticSlot* out)
{
    std::lock_guard<std::mutex> lock(g_slots_mu);
    StaticSlot& s = g_slots[device];
    if (!s.table) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_segs);
        if (e != cudaSuccess || !ptr) {
            set_error("cudaGetSymbolAddress(static segment table): %s", cudaGetErrorString(e));
            return DR_ERR_CUDA;
        }
        int rc = ensure_bulk_smem(device);  // an attribute of the kernels, not an allocation
        if (rc) return rc;
        int g2 = choose_grid(device, 2), g4 = choose_grid(device, 4);
        if (g2 <= 0 || g4 <= 0) {
            set_error("occupancy query failed");
            return DR_ERR_CUDA;
        }
        s.grid[0] = g2;
        s.grid[1] = g4;
        s.table = (DevSeg*)ptr;
    }
    *out = s;
    return DR_OK;
}

}  // namespace
}  // namespace dr

extern "C" int dr_reshard_static(const dr_plan* plan, const void* src_dev, uint64_t src_bytes, void* dst_dev,
                                 uint64_t dst_bytes, void* cuda_stream)
{
    using namespace dr;
    if (!plan || !src_dev || !dst_dev) {
        set_error("NULL plan or buffer");
        return DR_ERR_INVALID;
    }
    const uint64_t n_segs = plan->dev_segs.size();
    if (plan->fp8) {
        set_error("fp8 plans are not supported by the static entry point");
        return DR_ERR_UNSUPPORTED;
    }
    if (n_segs > kStaticMaxSegs) {
        set_error("plan has %llu segments; the static table holds at most %u (use dr_plan_create + dr_reshard)",
                  (unsigned long long)n_segs, kStaticMaxSegs);
        return DR_ERR_SIZE;
    }
    if (src_bytes < plan->info.src_bytes || dst_bytes < plan->info.dst_bytes) {
        set_error("buffer too small: have %llu / %llu bytes, need %llu / %llu", (unsigned long long)src_bytes,
                  (unsigned long long)dst_bytes, (unsigned long long)plan->info.src_bytes,
                  (unsigned long long)plan->info.dst_bytes);
        return DR_ERR_SIZE;
    }
    if (((uintptr_t)src_dev | (uintptr_t)dst_dev) & 15) {
        set_error("base pointers must be 16-byte aligned");
        return DR_ERR_ALIGN;
    }
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) {
        set_error("no current CUDA device");
        return DR_ERR_CUDA;
    }
    StaticSlot slot;
    int rc = static_setup(device, &slot);
    if (rc) return rc;
    const uint64_t n_tiles = plan->info.n_tiles;
    if (n_tiles == 0) return DR_OK;
    if (n_tiles > 0x7FFFFFFFull) {
        set_error("%llu tiles exceed the largest grid", (unsigned long long)n_tiles);
        return DR_ERR_UNSUPPORTED;
    }
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // The table is rewritten for every call, in stream order before the kernel that reads it.
    cudaError_t e = cudaMemcpyAsync(slot.table, plan->dev_segs.data(), n_segs * sizeof(DevSeg), cudaMemcpyHostToDevice, s);
    uint32_t* hints = (uint32_t*)((char*)slot.table + kStaticSegBytes);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(hints, plan->hints.data(), plan->hints.size() * sizeof(uint32_t), cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) {
        set_error("static table upload: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    char* f = (char*)src_dev;
    char* a = (char*)dst_dev;
    const int allow256 = (((uintptr_t)f | (uintptr_t)a) & 31) == 0;
    const int g = slot.grid[plan->elem_size == 2 ? 0 : 1];
    const uint64_t want = DR_GRID_MULT ? (uint64_t)g : (n_tiles + DR_TILES_PER_CTA - 1) / DR_TILES_PER_CTA;
    dim3 grid((unsigned)(n_tiles < want ? n_tiles : want)), block(kThreads);
#define DR_LAUNCH_S(ES, BULK)                                                                                   \
    reshard_kernel<ES, false, DR_BLOCKED, false, BULK><<<grid, block, (BULK) ? DR_DYN_SMEM : DR_OCC_SMEM, s>>>(    \
        slot.table, (uint32_t)n_segs, hints, plan->hint_shift, 0, n_tiles, f, a, allow256)
    const bool bulk = DR_BULK && plan->bulk_forward;
    if (plan->elem_size == 2) {
        if (bulk) DR_LAUNCH_S(2, true); else DR_LAUNCH_S(2, false);
    } else {
        if (bulk) DR_LAUNCH_S(4, true); else DR_LAUNCH_S(4, false);
    }
#undef DR_LAUNCH_S
    e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_error("reshard kernel launch: %s", cudaGetErrorString(e));
        return DR_ERR_CUDA;
    }
    return DR_OK;
}
