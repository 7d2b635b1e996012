// Bounded chunked host staging: a pinned ring of chunk slots, a copy stream and a relay stream,
// and worker threads that move chunks between the ring and a pageable host arena behind the pump.
// Every wait is a bounded host-side poll; there is no device-side waiting anywhere.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstdlib>
#include <cstring>
#include <exception>
#include <functional>
#include <string>
#include <thread>

#include "copy_pool.h"
#include "dr_internal.h"

namespace dr {

namespace {

using Clock = std::chrono::steady_clock;

double ms_since(Clock::time_point t0) { return std::chrono::duration<double, std::milli>(Clock::now() - t0).count(); }

// Rings up to this size are filled with ordinary (cached) stores on stage-in.
#ifndef DR_CACHED_RING_BYTES
#define DR_CACHED_RING_BYTES (64ull << 20)
#endif
constexpr uint64_t kCachedRingBytes = DR_CACHED_RING_BYTES;

// A single core cannot keep up with the host link; beyond 16 threads the copy is bound by memory, not cores.
// Two cores are left to the pump and to the driver's own thread: with a worker on every core the pump is
// descheduled between chunks and the link idles (measured on 16 cores, 16 x 4 MiB ring, stage-out: 14 workers
// 0.95 of the link, 16 workers 0.83).  DR_COPY_THREADS (1..64) overrides the count, read when a plan starts
// its workers.
unsigned default_copy_threads()
{
    if (const char* e = std::getenv("DR_COPY_THREADS")) {
        long v = std::strtol(e, nullptr, 10);
        if (v >= 1 && v <= 64) return (unsigned)v;
    }
    unsigned hw = std::thread::hardware_concurrency();
    return std::max(1u, std::min(16u, hw > 4 ? hw - 2 : hw));
}

}  // namespace

// Set by the deferred form's thread: where dr_stage_in announces, buffer by buffer, that a buffer is resident.
thread_local std::atomic<int>* tl_buffer_ready = nullptr;

struct Ring {
    cudaStream_t s_copy = nullptr, s_relay = nullptr;
    char* base = nullptr;  // pinned, at least slots * chunk bytes
    uint64_t capacity = 0; // bytes allocated at base
    uint64_t chunk = 0;
    uint32_t slots = 0;
    std::vector<cudaEvent_t> ev_copy, ev_relay;  // one per slot
    cudaEvent_t ev_entry = nullptr;              // recorded on the caller's stream when a call begins
    std::unique_ptr<Drainer> drainer;  // started by the first stage-out into a pageable arena
    std::unique_ptr<std::atomic<uint32_t>[]> pending;  // per slot: host-copy tasks of the chunk in it still to run
    uint32_t pending_slots = 0;
};

void ring_destroy(Ring* r)
{
    if (!r) return;
    if (r->s_copy) cudaStreamSynchronize(r->s_copy);
    if (r->s_relay) cudaStreamSynchronize(r->s_relay);
    r->drainer.reset();  // joins its thread; nothing is queued once a stage call has returned
    for (auto e : r->ev_copy) cudaEventDestroy(e);
    for (auto e : r->ev_relay) cudaEventDestroy(e);
    if (r->ev_entry) cudaEventDestroy(r->ev_entry);
    if (r->base) cudaFreeHost(r->base);
    if (r->s_copy) cudaStreamDestroy(r->s_copy);
    if (r->s_relay) cudaStreamDestroy(r->s_relay);
    delete r;
}

namespace {

struct Geometry {
    uint64_t total = 0, chunk = 0, n_chunks = 0;
    uint32_t slots = 0;
    uint64_t prefix[DR_MAX_STAGE_BUFS + 1] = {0};
    uint64_t host_at[DR_MAX_STAGE_BUFS] = {0};  // where buffer i rests inside the host arena
    bool scattered = false;                      // host positions differ from stream positions
};

bool is_pinned_host(const void* p);

// Chunk size a call gets when it names none and its bytes pass through the ring by DMA on one side and by DMA or
// the worker threads on the other (relay target, pageable arena): slots this small keep the ring inside the host's
// last-level cache, which is what makes that path fast (see the header).  Never more than the usual budget / 2.
constexpr uint64_t kAutoChunkOut = 4ull << 20, kAutoChunkIn = 8ull << 20, kAutoRingBytes = 64ull << 20;

int geometry(const dr_stage_desc* d, Geometry* g, bool out)
{
    if (!d || d->struct_size != sizeof(dr_stage_desc) || d->n_bufs == 0 || d->n_bufs > DR_MAX_STAGE_BUFS) {
        set_error("bad staging descriptor");
        return DR_ERR_INVALID;
    }
    for (uint32_t i = 0; i < d->n_bufs; ++i) {
        if (!d->dev_ptr[i] && d->bytes[i]) {
            set_error("NULL device buffer %u", i);
            return DR_ERR_INVALID;
        }
        g->prefix[i + 1] = g->prefix[i] + d->bytes[i];
    }
    g->total = g->prefix[d->n_bufs];
    g->scattered = (d->flags & DR_STAGE_HOST_OFFSETS) != 0;
    for (uint32_t i = 0; i < d->n_bufs; ++i) g->host_at[i] = g->scattered ? d->host_offset[i] : g->prefix[i];
    uint64_t budget = d->budget_bytes;
    g->chunk = d->chunk_bytes ? d->chunk_bytes : budget / 2 / 4096 * 4096;
    if (!d->chunk_bytes && !d->callback) {
        bool relay = false;
        for (uint32_t i = 0; out && i < d->n_bufs; ++i) relay |= d->relay_dev[i] != nullptr && d->bytes[i] != 0;
        const bool pageable = d->host_arena && !is_pinned_host(d->host_arena);
        const uint64_t small = out ? kAutoChunkOut : kAutoChunkIn;
        if ((relay || pageable) && g->chunk > small) {
            g->chunk = small;
            budget = std::min(budget, kAutoRingBytes);
        }
    }
    if (g->chunk == 0 || budget / g->chunk < 2) {
        set_error("budget %llu cannot hold two slots of %llu bytes", (unsigned long long)d->budget_bytes,
                  (unsigned long long)g->chunk);
        return DR_ERR_BUDGET;
    }
    g->slots = (uint32_t)std::min<uint64_t>(budget / g->chunk, 64);
    g->n_chunks = (g->total + g->chunk - 1) / g->chunk;
    return DR_OK;
}

int ensure_ring(dr_plan* p, const Geometry& g, bool need_memory, uint64_t budget)
{
    if (!p->ring) {
        Ring* r = new (std::nothrow) Ring();
        if (!r) return DR_ERR_NOMEM;
        p->ring = r;
        DR_CUDA(cudaStreamCreateWithFlags(&r->s_copy, cudaStreamNonBlocking));
        DR_CUDA(cudaStreamCreateWithFlags(&r->s_relay, cudaStreamNonBlocking));
        DR_CUDA(cudaEventCreateWithFlags(&r->ev_entry, cudaEventDisableTiming));
    }
    Ring* r = p->ring;
    while (r->ev_copy.size() < g.slots) {
        cudaEvent_t a, b;
        DR_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
        r->ev_copy.push_back(a);
        DR_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
        r->ev_relay.push_back(b);
    }
    // a ring that is large enough, and not larger than this call's budget, is kept and re-cut
    if (need_memory && (g.chunk * g.slots > r->capacity || r->capacity > budget)) {
        if (r->base) {
            DR_CUDA(cudaStreamSynchronize(r->s_copy));
            DR_CUDA(cudaStreamSynchronize(r->s_relay));
            cudaFreeHost(r->base);
            r->base = nullptr;
            r->capacity = 0;
        }
        DR_CUDA(cudaHostAlloc((void**)&r->base, g.chunk * g.slots, cudaHostAllocDefault));
        r->capacity = g.chunk * g.slots;
    }
    if (need_memory) {
        r->chunk = g.chunk;
        r->slots = g.slots;
    }
    return DR_OK;
}

// Worker threads and per-slot task counters for copies between the ring and a pageable arena.
int ensure_drainer(Ring* r, uint32_t slots)
{
    try {
        if (!r->drainer) r->drainer.reset(new Drainer(default_copy_threads()));
        if (r->pending_slots < slots) {
            r->pending.reset(new std::atomic<uint32_t>[slots]);
            r->pending_slots = slots;
        }
    } catch (const std::exception& e) {
        set_error("cannot start the host copy threads: %s", e.what());
        return DR_ERR_NOMEM;
    }
    for (uint32_t i = 0; i < slots; ++i) r->pending[i].store(0);
    return DR_OK;
}

// The plan's streams are non-blocking, so nothing orders them after the caller's work by itself: make them
// wait for the caller's event, or for everything enqueued so far on the caller's stream.
int order_after_caller(Ring* r, const dr_stage_desc* d)
{
    cudaEvent_t ev = (cudaEvent_t)d->wait_event;
    if (!ev) {
        if (d->flags & DR_STAGE_UNORDERED) return DR_OK;
        DR_CUDA(cudaEventRecord(r->ev_entry, (cudaStream_t)d->caller_stream));
        ev = r->ev_entry;
    }
    DR_CUDA(cudaStreamWaitEvent(r->s_copy, ev, 0));
    DR_CUDA(cudaStreamWaitEvent(r->s_relay, ev, 0));
    return DR_OK;
}

// Bounded wait for an event: poll, back off, give up at the deadline.
int wait_event(cudaEvent_t ev, Clock::time_point deadline)
{
    for (unsigned spins = 0;; ++spins) {
        cudaError_t e = cudaEventQuery(ev);
        if (e == cudaSuccess) return DR_OK;
        if (e != cudaErrorNotReady) {
            set_error("cudaEventQuery: %s", cudaGetErrorString(e));
            return DR_ERR_CUDA;
        }
        if (Clock::now() > deadline) {
            set_error("staging wait timed out");
            return DR_ERR_TIMEOUT;
        }
        if (spins < 200) std::this_thread::yield();
        else std::this_thread::sleep_for(std::chrono::microseconds(20));
    }
}

// Bounded drain of both streams on an error path, so that no copy still targets the ring or the caller's
// arena on return.  The bound is generous and independent of the caller's timeout: copies that were already
// enqueued cannot be cancelled, only waited for.
void drain(Ring* r)
{
    const auto deadline = Clock::now() + std::chrono::seconds(20);
    for (cudaStream_t s : {r->s_copy, r->s_relay})
        while (cudaStreamQuery(s) == cudaErrorNotReady && Clock::now() < deadline)
            std::this_thread::sleep_for(std::chrono::microseconds(50));
}

bool is_pinned_host(const void* p)
{
    cudaPointerAttributes a{};
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return a.type == cudaMemoryTypeHost;
}

int check_common(dr_plan* p, const dr_stage_desc* d, const Geometry& g, bool out)
{
    if (p->host_only) {
        set_error("host-only plan cannot stage");
        return DR_ERR_STATE;
    }
    // a callback takes everything and excludes the rest; otherwise every non-empty buffer needs a place to go:
    // its relay target (stage-out only) or the host arena
    bool any_relay = false, any_unplaced = false;
    for (uint32_t i = 0; i < d->n_bufs; ++i) {
        if (out && d->relay_dev[i]) any_relay = true;
        else if (d->bytes[i] && !d->host_arena) any_unplaced = true;
    }
    if (d->callback ? (d->host_arena != nullptr || any_relay) : any_unplaced) {
        set_error(d->callback ? "a callback excludes host_arena and relay_dev"
                              : "a buffer has neither a relay target nor a host arena to go to");
        return DR_ERR_INVALID;
    }
    if (g.scattered && !d->host_arena) {
        set_error("DR_STAGE_HOST_OFFSETS needs a host arena");
        return DR_ERR_INVALID;
    }
    if (d->host_arena && !g.scattered && d->host_arena_bytes < g.total) {
        set_error("host arena holds %llu bytes, stream is %llu", (unsigned long long)d->host_arena_bytes,
                  (unsigned long long)g.total);
        return DR_ERR_SIZE;
    }
    if (g.scattered) {
        auto rests_on_host = [&](uint32_t i) { return d->bytes[i] && !(out && d->relay_dev[i]); };
        for (uint32_t i = 0; i < d->n_bufs; ++i) {
            if (!rests_on_host(i)) continue;
            if (g.host_at[i] + d->bytes[i] > d->host_arena_bytes) {
                set_error("buffer %u does not fit the host arena at its offset", i);
                return DR_ERR_SIZE;
            }
            for (uint32_t j = 0; j < i; ++j)
                if (rests_on_host(j) && g.host_at[i] < g.host_at[j] + d->bytes[j] && g.host_at[j] < g.host_at[i] + d->bytes[i]) {
                    set_error("host regions of buffers %u and %u overlap", j, i);
                    return DR_ERR_INVALID;
                }
        }
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != p->device) {
        set_error("current device differs from the plan's device");
        return DR_ERR_STATE;
    }
    return DR_OK;
}

}  // namespace
}  // namespace dr

using namespace dr;

extern "C" int dr_stage_out(dr_plan* plan, const dr_stage_desc* d, dr_stage_stats* stats)
{
    if (!plan) {
        set_error("NULL plan");
        return DR_ERR_INVALID;
    }
    Geometry g;
    int rc = geometry(d, &g, true);
    if (rc) return rc;
    if ((rc = check_common(plan, d, g, true))) return rc;
    std::lock_guard<std::mutex> lock(plan->stage_mu);
    // Where each buffer goes: to its relay target (device -> ring slot -> device), or to the host arena (straight
    // into a pinned arena, through the ring and the host copy threads into a pageable one); or everything to the
    // callback.  A call may mix relay and arena buffers: a rank whose new shard is partly on this GPU already
    // relays that part and rests the remainder on the host in one pass.
    bool to_relay[DR_MAX_STAGE_BUFS] = {false};
    bool any_relay = false, any_host = false;
    for (uint32_t b = 0; b < d->n_bufs && !d->callback; ++b) {
        to_relay[b] = d->relay_dev[b] != nullptr;
        if (d->bytes[b] == 0) continue;
        any_relay |= to_relay[b];
        any_host |= !to_relay[b];
    }
    const bool pinned_arena = any_host && is_pinned_host(d->host_arena);  // DMA straight into the arena
    const bool via_drainer = any_host && !pinned_arena;                   // pageable arena: drainer thread copies out
    const bool need_ring = d->callback || any_relay || via_drainer;
    if ((rc = ensure_ring(plan, g, need_ring, d->budget_bytes))) return rc;
    Ring* r = plan->ring;
    const auto t0 = Clock::now();
    const auto limit = std::chrono::milliseconds(d->timeout_ms ? d->timeout_ms : 60000);
    dr_stage_stats st{};
    st.n_chunks = g.n_chunks;
    st.chunks_done = std::min<uint64_t>(d->first_chunk, g.n_chunks);
    st.pinned_high_water_bytes = need_ring ? g.chunk * g.slots : 0;
    if ((rc = order_after_caller(r, d))) return rc;

    // ring slot of chunk k (unused when every chunk is copied straight into a pinned arena)
    auto slot_ptr = [&](uint64_t k) -> char* { return r->base + (k % g.slots) * g.chunk; };
    // enqueue the copies of chunk k: one per buffer it touches
    auto issue = [&](uint64_t k) -> int {
        uint64_t lo = k * g.chunk, hi = std::min(lo + g.chunk, g.total);
        uint32_t s = (uint32_t)(k % g.slots);
        char* host = need_ring ? slot_ptr(k) : nullptr;
        for (uint32_t b = 0; b < d->n_bufs; ++b) {
            uint64_t a = std::max(lo, g.prefix[b]), e = std::min(hi, g.prefix[b + 1]);
            if (a >= e) continue;
            const bool straight = !d->callback && !to_relay[b] && pinned_arena;
            char* to = straight ? (char*)d->host_arena + g.host_at[b] + (a - g.prefix[b]) : host + (a - lo);
            DR_CUDA(cudaMemcpyAsync(to, (const char*)d->dev_ptr[b] + (a - g.prefix[b]), e - a, cudaMemcpyDeviceToHost,
                                    r->s_copy));
        }
        DR_CUDA(cudaEventRecord(r->ev_copy[s], r->s_copy));
        if (any_relay) {
            DR_CUDA(cudaStreamWaitEvent(r->s_relay, r->ev_copy[s], 0));
            for (uint32_t b = 0; b < d->n_bufs; ++b) {
                uint64_t a = std::max(lo, g.prefix[b]), e = std::min(hi, g.prefix[b + 1]);
                if (a >= e || !to_relay[b]) continue;
                DR_CUDA(cudaMemcpyAsync((char*)d->relay_dev[b] + (a - g.prefix[b]), host + (a - lo), e - a,
                                        cudaMemcpyHostToDevice, r->s_relay));
            }
            DR_CUDA(cudaEventRecord(r->ev_relay[s], r->s_relay));
        }
        return DR_OK;
    };
    // A pageable arena is filled by the drainer's worker threads: the pump hands them a chunk as soon as the chunk
    // has arrived in its ring slot and goes on issuing copies; the slot is free again once the chunk is copied out.
    if (via_drainer && (rc = ensure_drainer(r, g.slots))) return rc;
    uint64_t handed = 0;  // chunks given to the drainer by this call

    // wait for chunk k and hand it to the sink
    auto complete = [&](uint64_t k) -> int {
        uint64_t lo = k * g.chunk, n = std::min(lo + g.chunk, g.total) - lo;
        uint32_t s = (uint32_t)(k % g.slots);
        int w = wait_event(r->ev_copy[s], Clock::now() + limit);
        if (w == DR_OK && any_relay) w = wait_event(r->ev_relay[s], Clock::now() + limit);
        if (w) return w;
        if (d->callback) {
            if (d->callback(d->user, k, lo, slot_ptr(k), n)) {
                set_error("chunk callback failed at chunk %llu", (unsigned long long)k);
                return DR_ERR_SINK;
            }
        } else if (via_drainer) {
            Drainer::Part parts[DR_MAX_STAGE_BUFS];
            unsigned np = 0;
            for (uint32_t b = 0; b < d->n_bufs; ++b) {  // one copy per arena-bound buffer the chunk touches
                uint64_t a = std::max(lo, g.prefix[b]), e = std::min(lo + n, g.prefix[b + 1]);
                if (a < e && !to_relay[b])
                    parts[np++] = Drainer::Part{(char*)d->host_arena + g.host_at[b] + (a - g.prefix[b]), slot_ptr(k) + (a - lo),
                                                e - a};
            }
            r->drainer->submit(parts, np, &r->pending[s]);  // possibly nothing to copy (a chunk of relay bytes only)
            ++handed;
            return DR_OK;  // counted as done once the workers have copied it out
        }
        st.bytes += n;
        return DR_OK;
    };
    auto chunk_bytes_of = [&](uint64_t k) { return std::min((k + 1) * g.chunk, g.total) - k * g.chunk; };

    const uint64_t first = st.chunks_done;
    uint64_t next_issue = first, next_done = first;  // next_done: next chunk whose device-to-host copy is awaited
    if (!via_drainer) {
        while (rc == DR_OK && next_done < g.n_chunks) {
            while (rc == DR_OK && next_issue < g.n_chunks && next_issue - next_done < g.slots) rc = issue(next_issue++);
            if (rc == DR_OK && (rc = complete(next_done)) == DR_OK) st.chunks_done = ++next_done;
        }
    } else {
        uint64_t out = first;  // chunks below this index rest in the arena; their slots are free
        auto refresh = [&] {   // chunks leave in order: chunk `out` is out once it was handed over and its tasks are done
            while (out < first + handed && r->pending[out % g.slots].load(std::memory_order_acquire) == 0)
                st.bytes += chunk_bytes_of(out++);
            st.chunks_done = out;
        };
        while (rc == DR_OK && out < g.n_chunks) {
            refresh();
            while (rc == DR_OK && next_issue < g.n_chunks && next_issue - out < g.slots) rc = issue(next_issue++);
            if (rc != DR_OK || out >= g.n_chunks) break;
            if (next_done < next_issue) {
                if ((rc = complete(next_done)) == DR_OK) ++next_done;
            } else {  // every issued chunk is with the workers: wait for the oldest slot to come back
                if (!r->drainer->wait_zero(&r->pending[out % g.slots], Clock::now() + limit)) {
                    set_error("staging wait timed out (host copy)");
                    rc = DR_ERR_TIMEOUT;
                }
            }
        }
        // whatever happened, no host copy of this call may still be running when it returns
        for (uint64_t k = out; k < first + handed; ++k)
            r->drainer->wait_zero(&r->pending[k % g.slots], Clock::now() + std::chrono::seconds(60));
        refresh();
    }
    if (rc) drain(r);
    if (d->done_event) cudaEventRecord((cudaEvent_t)d->done_event, any_relay ? r->s_relay : r->s_copy);
    st.elapsed_ms = ms_since(t0);
    st.link_gbs = st.elapsed_ms > 0 ? (double)st.bytes / st.elapsed_ms * 1e-6 : 0;
    if (stats) *stats = st;
    return rc;
}

extern "C" int dr_stage_in(dr_plan* plan, const dr_stage_desc* d, dr_stage_stats* stats)
{
    if (!plan) {
        set_error("NULL plan");
        return DR_ERR_INVALID;
    }
    Geometry g;
    int rc = geometry(d, &g, false);
    if (rc) return rc;
    if ((rc = check_common(plan, d, g, false))) return rc;
    {
        uint32_t seen = 0;
        for (uint32_t i = 0; i < d->n_bufs; ++i)
            if (d->order[i] < d->n_bufs) seen |= 1u << d->order[i];
        if (seen != (1u << d->n_bufs) - 1) {
            set_error("order[] must be a permutation of 0..n_bufs-1");
            return DR_ERR_INVALID;
        }
    }
    std::lock_guard<std::mutex> lock(plan->stage_mu);
    const bool direct = !d->callback && is_pinned_host(d->host_arena);
    if ((rc = ensure_ring(plan, g, !direct, d->budget_bytes))) return rc;
    Ring* r = plan->ring;
    const auto t0 = Clock::now();
    const auto limit = std::chrono::milliseconds(d->timeout_ms ? d->timeout_ms : 60000);

    struct Piece {
        uint32_t buf;
        bool last;
        uint64_t pos, n;
    };
    std::vector<Piece> pieces;
    for (uint32_t o = 0; o < d->n_bufs; ++o) {
        uint32_t b = d->order[o];
        for (uint64_t pos = 0; pos < d->bytes[b]; pos += g.chunk) {
            uint64_t n = std::min(g.chunk, d->bytes[b] - pos);
            pieces.push_back(Piece{b, pos + n == d->bytes[b], pos, n});
        }
    }
    dr_stage_stats st{};
    st.n_chunks = pieces.size();
    st.chunks_done = std::min<uint64_t>(d->first_chunk, pieces.size());
    st.pinned_high_water_bytes = direct ? 0 : g.chunk * g.slots;
    if ((rc = order_after_caller(r, d))) return rc;
    if (tl_buffer_ready) {  // buffers this call has nothing to do for: empty, or complete before first_chunk
        bool pending[DR_MAX_STAGE_BUFS] = {false};
        for (uint64_t i = st.chunks_done; i < pieces.size(); ++i) pending[pieces[i].buf] = true;
        for (uint32_t b = 0; b < d->n_bufs; ++b)
            if (!pending[b]) tl_buffer_ready[b].store(1, std::memory_order_release);
    }

    auto issue = [&](uint64_t i) -> int {
        const Piece& pc = pieces[i];
        uint32_t s = (uint32_t)(i % g.slots);
        uint64_t off = g.prefix[pc.buf] + pc.pos;            // position in the stream (what a callback sees)
        uint64_t at = g.host_at[pc.buf] + pc.pos;            // position in the host arena
        const char* host;
        if (direct) {
            host = (const char*)d->host_arena + at;
        } else {
            char* slot = r->base + (uint64_t)s * g.chunk;
            if (d->callback) {
                if (d->callback(d->user, i, off, slot, pc.n)) {
                    set_error("chunk callback failed at piece %llu", (unsigned long long)i);
                    return DR_ERR_SINK;
                }
            }  // (a pageable arena does not come here: its slots are filled by the worker threads, see below)
            host = slot;
        }
        DR_CUDA(cudaMemcpyAsync((char*)d->dev_ptr[pc.buf] + pc.pos, host, pc.n, cudaMemcpyHostToDevice, r->s_copy));
        DR_CUDA(cudaEventRecord(r->ev_copy[s], r->s_copy));
        if (pc.last && d->ready_events[pc.buf]) DR_CUDA(cudaEventRecord((cudaEvent_t)d->ready_events[pc.buf], r->s_copy));
        return DR_OK;
    };
    auto complete = [&](uint64_t i) -> int {
        int w = wait_event(r->ev_copy[i % g.slots], Clock::now() + limit);
        if (w) return w;
        st.bytes += pieces[i].n;
        if (pieces[i].last) {
            st.ready_ms[pieces[i].buf] = ms_since(t0);
            if (tl_buffer_ready) tl_buffer_ready[pieces[i].buf].store(1, std::memory_order_release);
        }
        return DR_OK;
    };

    uint64_t next_issue = st.chunks_done, next_done = st.chunks_done;
    const bool via_filler = !direct && !d->callback;  // pageable arena: worker threads fill the ring slots
    if (!via_filler) {
        while (rc == DR_OK && next_done < pieces.size()) {
            if (next_issue < pieces.size() && next_issue - next_done < g.slots) {
                if ((rc = issue(next_issue)) == DR_OK) ++next_issue;  // a piece whose source failed was not issued
            } else if ((rc = complete(next_done)) == DR_OK) {
                st.chunks_done = ++next_done;
            }
        }
    } else if ((rc = ensure_drainer(r, g.slots)) == DR_OK) {
        // Three cursors: pieces below next_fill have been given to the workers (pageable arena -> ring slot), pieces
        // below next_issue are on their way to the device, pieces below next_done have arrived.  A slot is refilled
        // once its previous piece has arrived.  A small ring is filled with ordinary stores, so that the device can
        // read it from the last-level cache; a large one with non-temporal stores.
        const bool cached = g.chunk * g.slots <= kCachedRingBytes;
        uint64_t next_fill = next_issue;
        auto fill = [&](uint64_t i) {
            const Piece& pc = pieces[i];
            const uint32_t s = (uint32_t)(i % g.slots);
            Drainer::Part part{r->base + (uint64_t)s * g.chunk, (const char*)d->host_arena + g.host_at[pc.buf] + pc.pos, pc.n, cached};
            r->drainer->submit(&part, 1, &r->pending[s]);
        };
        auto send = [&](uint64_t i) -> int {
            const Piece& pc = pieces[i];
            const uint32_t s = (uint32_t)(i % g.slots);
            DR_CUDA(cudaMemcpyAsync((char*)d->dev_ptr[pc.buf] + pc.pos, r->base + (uint64_t)s * g.chunk, pc.n,
                                    cudaMemcpyHostToDevice, r->s_copy));
            DR_CUDA(cudaEventRecord(r->ev_copy[s], r->s_copy));
            if (pc.last && d->ready_events[pc.buf])
                DR_CUDA(cudaEventRecord((cudaEvent_t)d->ready_events[pc.buf], r->s_copy));
            return DR_OK;
        };
        while (rc == DR_OK && next_done < pieces.size()) {
            // retire arrivals without blocking, so that their slots can be refilled at once
            while (next_done < next_issue && cudaEventQuery(r->ev_copy[next_done % g.slots]) == cudaSuccess) {
                st.bytes += pieces[next_done].n;
                if (pieces[next_done].last) {
                    st.ready_ms[pieces[next_done].buf] = ms_since(t0);
                    if (tl_buffer_ready) tl_buffer_ready[pieces[next_done].buf].store(1, std::memory_order_release);
                }
                st.chunks_done = ++next_done;
            }
            while (next_fill < pieces.size() && next_fill - next_done < g.slots) fill(next_fill++);
            while (rc == DR_OK && next_issue < next_fill &&
                   r->pending[next_issue % g.slots].load(std::memory_order_acquire) == 0)
                if ((rc = send(next_issue)) == DR_OK) ++next_issue;
            if (rc != DR_OK || next_done >= pieces.size()) break;
            if (next_issue < next_fill) {  // a fill is under way: it ends within milliseconds
                if (!r->drainer->wait_zero(&r->pending[next_issue % g.slots], Clock::now() + limit)) {
                    set_error("staging wait timed out (host copy)");
                    rc = DR_ERR_TIMEOUT;
                }
            } else if ((rc = complete(next_done)) == DR_OK) {
                st.chunks_done = ++next_done;
            }
        }
        for (uint64_t k = next_issue; k < next_fill; ++k)  // no host copy of this call may outlive it
            r->drainer->wait_zero(&r->pending[k % g.slots], Clock::now() + std::chrono::seconds(60));
    }
    if (rc) {
        drain(r);
        // pieces that were on their way when the call failed have landed during the drain: they count as done
        while (next_done < next_issue && cudaEventQuery(r->ev_copy[next_done % g.slots]) == cudaSuccess) {
            st.bytes += pieces[next_done].n;
            if (pieces[next_done].last) {
                st.ready_ms[pieces[next_done].buf] = ms_since(t0);
                if (tl_buffer_ready) tl_buffer_ready[pieces[next_done].buf].store(1, std::memory_order_release);
            }
            st.chunks_done = ++next_done;
        }
    }
    if (d->done_event) cudaEventRecord((cudaEvent_t)d->done_event, r->s_copy);
    st.elapsed_ms = ms_since(t0);
    st.link_gbs = st.elapsed_ms > 0 ? (double)st.bytes / st.elapsed_ms * 1e-6 : 0;
    if (stats) *stats = st;
    return rc;
}

// ---- deferred form: the same pump on a thread of the library's own --------------------------------------------
struct dr_stage_job {
    std::thread th;
    dr_plan* plan = nullptr;
    dr_stage_desc desc{};
    int direction = 0;
    dr_stage_stats stats{};
    int rc = DR_OK;
    std::string err;
    std::atomic<int> done{0};
    std::atomic<int> ready[DR_MAX_STAGE_BUFS];  // stage-in: buffer i is resident (its last copy has completed)
    cudaEvent_t entry = nullptr;  // the ordering point, recorded on the caller's stream by dr_stage_begin
};

extern "C" int dr_stage_begin(dr_plan* plan, const dr_stage_desc* d, int direction, dr_stage_job** out)
{
    if (!plan || !out || (direction != DR_STAGE_DIR_OUT && direction != DR_STAGE_DIR_IN)) {
        set_error("NULL plan or job pointer, or unknown direction");
        return DR_ERR_INVALID;
    }
    *out = nullptr;
    Geometry g;
    int rc = geometry(d, &g, direction == DR_STAGE_DIR_OUT);
    if (rc) return rc;
    if ((rc = check_common(plan, d, g, direction == DR_STAGE_DIR_OUT))) return rc;
    dr_stage_job* job = new (std::nothrow) dr_stage_job();
    if (!job) return DR_ERR_NOMEM;
    for (auto& r : job->ready) r.store(0);
    job->plan = plan;
    job->desc = *d;
    job->direction = direction;
    // the pump would take its ordering point when it starts, some time after this call has returned: take it now
    if (!d->wait_event && !(d->flags & DR_STAGE_UNORDERED)) {
        cudaError_t e = cudaEventCreateWithFlags(&job->entry, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventRecord(job->entry, (cudaStream_t)d->caller_stream);
        if (e != cudaSuccess) {
            set_error("ordering event: %s", cudaGetErrorString(e));
            if (job->entry) cudaEventDestroy(job->entry);
            delete job;
            return DR_ERR_CUDA;
        }
        job->desc.wait_event = job->entry;
    }
    try {
        job->th = std::thread([job] {
            if (cudaSetDevice(job->plan->device) != cudaSuccess) {
                job->rc = DR_ERR_CUDA;
                job->err = "cudaSetDevice on the staging thread failed";
            } else {
                tl_buffer_ready = job->ready;
                job->rc = job->direction == DR_STAGE_DIR_OUT ? dr_stage_out(job->plan, &job->desc, &job->stats)
                                                             : dr_stage_in(job->plan, &job->desc, &job->stats);
                tl_buffer_ready = nullptr;
                if (job->rc) job->err = dr_last_error();
            }
            job->done.store(1, std::memory_order_release);
        });
    } catch (const std::exception& e) {
        set_error("cannot start the staging thread: %s", e.what());
        if (job->entry) cudaEventDestroy(job->entry);
        delete job;
        return DR_ERR_NOMEM;
    }
    *out = job;
    return DR_OK;
}

extern "C" int dr_stage_poll(const dr_stage_job* job, int* done)
{
    if (!job || !done) {
        set_error("NULL job or result pointer");
        return DR_ERR_INVALID;
    }
    *done = job->done.load(std::memory_order_acquire);
    return DR_OK;
}

extern "C" int dr_stage_wait_buffer(dr_stage_job* job, uint32_t buffer, uint32_t timeout_ms)
{
    if (!job || buffer >= DR_MAX_STAGE_BUFS || buffer >= job->desc.n_bufs || job->direction != DR_STAGE_DIR_IN) {
        set_error("NULL job, buffer index out of range, or not a stage-in job");
        return DR_ERR_INVALID;
    }
    const auto deadline = Clock::now() + std::chrono::milliseconds(timeout_ms ? timeout_ms : 60000);
    for (unsigned spins = 0;; ++spins) {
        if (job->ready[buffer].load(std::memory_order_acquire)) return DR_OK;
        if (job->done.load(std::memory_order_acquire)) {  // the pump has returned without this buffer: it failed
            if (job->ready[buffer].load(std::memory_order_acquire)) return DR_OK;
            set_error("the stage-in ended before buffer %u was resident: %s", buffer, job->err.c_str());
            return job->rc ? job->rc : DR_ERR_STATE;
        }
        if (Clock::now() > deadline) {
            set_error("buffer %u not resident within the time given", buffer);
            return DR_ERR_TIMEOUT;
        }
        if (spins < 200) std::this_thread::yield();
        else std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
}

extern "C" int dr_stage_end(dr_stage_job* job, dr_stage_stats* stats)
{
    if (!job) {
        set_error("NULL job");
        return DR_ERR_INVALID;
    }
    if (job->th.joinable()) job->th.join();
    if (job->entry) cudaEventDestroy(job->entry);
    if (stats) *stats = job->stats;
    const int rc = job->rc;
    if (rc) set_error("%s", job->err.c_str());
    delete job;
    return rc;
}

extern "C" int dr_host_copy(void* dst_host, const void* src_host, uint64_t n_bytes, uint32_t threads)
{
    if (!dst_host || !src_host) {
        set_error("NULL host pointer");
        return DR_ERR_INVALID;
    }
    try {  // the engine's own workers and task size, on one copy
        Drainer workers(threads ? threads : default_copy_threads());
        std::atomic<uint32_t> pending{0};
        Drainer::Part part{(char*)dst_host, (const char*)src_host, n_bytes, false};
        workers.submit(&part, 1, &pending);
        while (!workers.wait_zero(&pending, Clock::now() + std::chrono::seconds(60))) {
        }
    } catch (const std::exception& e) {
        set_error("cannot start the host copy threads: %s", e.what());
        return DR_ERR_NOMEM;
    }
    return DR_OK;
}
