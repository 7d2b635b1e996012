// Streamed repack: H2D chunks of the flat source, one repack kernel per chunk, D2H of arena ranges that
// have become final -- three streams tied together by events, enqueued up front, awaited once.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <new>
#include <thread>

#include "dr_internal.h"

namespace dr {

struct ChunkTables {
    uint64_t seg_off = 0, hint_off = 0;  // element offsets into the device pools
    uint32_t n_segs = 0, hint_shift = 0;
    uint64_t n_tiles = 0;
    uint64_t final_below = 0;  // after this chunk's kernel, arena bytes below this offset never change again
};

struct Stream {
    uint64_t chunk_bytes = 0;
    std::vector<ChunkTables> chunks;
    DevSeg* d_segs = nullptr;
    uint32_t* d_hints = nullptr;
    cudaStream_t s_h2d = nullptr, s_kernel = nullptr, s_d2h = nullptr;
    std::vector<cudaEvent_t> ev_arrived, ev_done;  // per window slot
    cudaEvent_t ev_first = nullptr, ev_last_kernel = nullptr, ev_last_copy = nullptr;
};

void stream_destroy(Stream* s)
{
    if (!s) return;
    for (cudaStream_t st : {s->s_h2d, s->s_kernel, s->s_d2h})
        if (st) {
            cudaStreamSynchronize(st);
            cudaStreamDestroy(st);
        }
    for (auto e : s->ev_arrived) cudaEventDestroy(e);
    for (auto e : s->ev_done) cudaEventDestroy(e);
    for (cudaEvent_t e : {s->ev_first, s->ev_last_kernel, s->ev_last_copy})
        if (e) cudaEventDestroy(e);
    if (s->d_segs) cudaFree(s->d_segs);
    if (s->d_hints) cudaFree(s->d_hints);
    delete s;
}

namespace {

// Per-chunk tables for a given chunk size, compiled once and kept on the device.
int prepare(dr_plan* p, uint64_t chunk_bytes, uint32_t slots)
{
    if (!p->stream) {
        p->stream = new (std::nothrow) Stream();
        if (!p->stream) return DR_ERR_NOMEM;
        Stream* s = p->stream;
        DR_CUDA(cudaStreamCreateWithFlags(&s->s_h2d, cudaStreamNonBlocking));
        DR_CUDA(cudaStreamCreateWithFlags(&s->s_kernel, cudaStreamNonBlocking));
        DR_CUDA(cudaStreamCreateWithFlags(&s->s_d2h, cudaStreamNonBlocking));
        DR_CUDA(cudaEventCreateWithFlags(&s->ev_first, cudaEventDisableTiming));
        DR_CUDA(cudaEventCreateWithFlags(&s->ev_last_kernel, cudaEventDisableTiming));
        DR_CUDA(cudaEventCreateWithFlags(&s->ev_last_copy, cudaEventDisableTiming));
    }
    Stream* s = p->stream;
    while (s->ev_arrived.size() < slots) {
        cudaEvent_t a, b;
        DR_CUDA(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
        s->ev_arrived.push_back(a);
        DR_CUDA(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
        s->ev_done.push_back(b);
    }
    if (s->chunk_bytes == chunk_bytes && !s->chunks.empty()) return DR_OK;

    const uint64_t chunk_elems = chunk_bytes / 4, src_elems = p->info.src_bytes / 4;
    const uint64_t n_chunks = (src_elems + chunk_elems - 1) / chunk_elems;
    std::vector<DevSeg> all_segs;
    std::vector<uint32_t> all_hints;
    std::vector<ChunkTables> chunks(n_chunks);
    std::vector<uint64_t> lowest(n_chunks + 1, p->info.dst_bytes);  // lowest arena byte chunk k writes
    for (uint64_t k = 0; k < n_chunks; ++k) {
        const uint64_t lo = k * chunk_elems, hi = std::min(lo + chunk_elems, src_elems);
        std::vector<HostSeg> segs = window_segments(p->segs, lo, hi, p->elem_size);
        Tables tb;
        int rc = build_tables(segs, &tb);
        if (rc) return rc;
        ChunkTables& c = chunks[k];
        c.seg_off = all_segs.size();
        c.hint_off = all_hints.size();
        c.n_segs = (uint32_t)tb.segs.size();
        c.hint_shift = tb.hint_shift;
        c.n_tiles = tb.n_tiles;
        all_segs.insert(all_segs.end(), tb.segs.begin(), tb.segs.end());
        all_hints.insert(all_hints.end(), tb.hints.begin(), tb.hints.end());
        for (const HostSeg& g : segs) lowest[k] = std::min(lowest[k], g.dst_off);
    }
    // arena bytes below min(lowest[j], j > k) are final once chunk k has been repacked
    uint64_t run = p->info.dst_bytes;
    for (uint64_t k = n_chunks; k-- > 0;) {
        chunks[k].final_below = run;
        run = std::min(run, lowest[k]);
    }
    if (s->d_segs) cudaFree(s->d_segs);
    if (s->d_hints) cudaFree(s->d_hints);
    s->d_segs = nullptr;
    s->d_hints = nullptr;
    s->chunks.clear();
    DR_CUDA(cudaMalloc((void**)&s->d_segs, std::max<size_t>(all_segs.size(), 1) * sizeof(DevSeg)));
    DR_CUDA(cudaMalloc((void**)&s->d_hints, std::max<size_t>(all_hints.size(), 1) * sizeof(uint32_t)));
    DR_CUDA(cudaMemcpy(s->d_segs, all_segs.data(), all_segs.size() * sizeof(DevSeg), cudaMemcpyHostToDevice));
    DR_CUDA(cudaMemcpy(s->d_hints, all_hints.data(), all_hints.size() * sizeof(uint32_t), cudaMemcpyHostToDevice));
    s->chunks.swap(chunks);
    s->chunk_bytes = chunk_bytes;
    return DR_OK;
}

}  // namespace
}  // namespace dr

using namespace dr;

extern "C" int dr_reshard_stream(dr_plan* plan, const dr_stream_desc* d, dr_stream_stats* stats)
{
    if (!plan || !d || d->struct_size != sizeof(dr_stream_desc) || !d->host_src || !d->dst_dev || !d->window_dev) {
        set_error("bad stream descriptor");
        return DR_ERR_INVALID;
    }
    if (plan->host_only) {
        set_error("host-only plan cannot launch");
        return DR_ERR_STATE;
    }
    if (plan->fp8) {
        set_error("fp8 plans cannot be streamed: a block needs all of its source rows");
        return DR_ERR_UNSUPPORTED;
    }
    if (d->host_src_bytes < plan->info.src_bytes || d->dst_bytes < plan->info.dst_bytes ||
        (d->host_dst && d->host_dst_bytes < plan->info.dst_bytes)) {
        set_error("a buffer is smaller than the plan needs");
        return DR_ERR_SIZE;
    }
    if (((uintptr_t)d->host_src | (uintptr_t)d->dst_dev | (uintptr_t)d->window_dev | (uintptr_t)d->host_dst) & 31) {
        set_error("pointers must be 32-byte aligned");
        return DR_ERR_ALIGN;
    }
    // no chunk size given: half the window, but not more than 32 MiB: small chunks start the pipeline early and
    // interleave the copy back with the copy in more finely (measured on the Qwen3-8B shape with the result copied
    // back to the host: 616 ms with 32 MiB chunks, 621 / 625 / 630 / 632 ms with 64 / 128 / 256 / 512 MiB)
    const uint64_t chunk = d->chunk_bytes ? d->chunk_bytes : std::min<uint64_t>(d->window_bytes / 2 / 4096 * 4096, 32ull << 20);
    if (chunk % 32) {
        set_error("chunk_bytes %llu is not a multiple of 32", (unsigned long long)chunk);
        return DR_ERR_INVALID;
    }
    if (chunk == 0 || d->window_bytes / chunk < 2) {
        set_error("window of %llu bytes cannot hold two chunks of %llu", (unsigned long long)d->window_bytes,
                  (unsigned long long)chunk);
        return DR_ERR_BUDGET;
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != plan->device) {
        set_error("current device differs from the plan's device");
        return DR_ERR_STATE;
    }
    std::lock_guard<std::mutex> lock(plan->stage_mu);
    const uint32_t slots = (uint32_t)std::min<uint64_t>(d->window_bytes / chunk, 16);
    int rc = prepare(plan, chunk, slots);
    if (rc) return rc;
    Stream* s = plan->stream;
    const auto t0 = std::chrono::steady_clock::now();
    dr_stream_stats st{};
    st.n_chunks = s->chunks.size();

    // Everything is enqueued up front; a failure stops the enqueueing, and what was already enqueued is still
    // waited for below.
    auto enqueue = [&]() -> int {
        uint64_t copied_below = 0;  // arena bytes already on their way to host_dst
        // The three streams are non-blocking: order them after the caller's event, or after everything the
        // caller has enqueued so far on its stream (a fill of the arena or the window must not land later).
        cudaEvent_t after = (cudaEvent_t)d->wait_event;
        if (!after && !(d->flags & DR_STREAM_UNORDERED)) {
            DR_CUDA(cudaEventRecord(s->ev_first, (cudaStream_t)d->caller_stream));
            after = s->ev_first;
        }
        if (after)
            for (cudaStream_t q : {s->s_h2d, s->s_kernel, s->s_d2h}) DR_CUDA(cudaStreamWaitEvent(q, after, 0));
        for (uint64_t k = 0; k < s->chunks.size(); ++k) {
            const ChunkTables& c = s->chunks[k];
            const uint32_t slot = (uint32_t)(k % slots);
            const uint64_t lo = k * chunk, n = std::min(chunk, plan->info.src_bytes - lo);
            char* win = (char*)d->window_dev + (uint64_t)slot * chunk;
            if (k >= slots) DR_CUDA(cudaStreamWaitEvent(s->s_h2d, s->ev_done[slot], 0));  // the slot's previous kernel
            DR_CUDA(cudaMemcpyAsync(win, (const char*)d->host_src + lo, n, cudaMemcpyHostToDevice, s->s_h2d));
            DR_CUDA(cudaEventRecord(s->ev_arrived[slot], s->s_h2d));
            st.h2d_bytes += n;
            DR_CUDA(cudaStreamWaitEvent(s->s_kernel, s->ev_arrived[slot], 0));
            int krc = launch_forward_tables(plan->elem_size, s->d_segs + c.seg_off, c.n_segs, s->d_hints + c.hint_off,
                                            c.hint_shift, c.n_tiles, win, d->dst_dev, s->s_kernel, plan->bulk_forward);
            if (krc) return krc;
            if (c.n_tiles) ++st.kernels;
            DR_CUDA(cudaEventRecord(s->ev_done[slot], s->s_kernel));
            if (d->host_dst && c.final_below > copied_below) {
                DR_CUDA(cudaStreamWaitEvent(s->s_d2h, s->ev_done[slot], 0));
                DR_CUDA(cudaMemcpyAsync((char*)d->host_dst + copied_below, (const char*)d->dst_dev + copied_below,
                                        c.final_below - copied_below, cudaMemcpyDeviceToHost, s->s_d2h));
                st.d2h_bytes += c.final_below - copied_below;
                copied_below = c.final_below;
            }
        }
        if (d->done_event) {  // after the last kernel (s_kernel) and the last copy back (s_d2h)
            DR_CUDA(cudaEventRecord(s->ev_last_kernel, s->s_kernel));
            DR_CUDA(cudaStreamWaitEvent(s->s_d2h, s->ev_last_kernel, 0));
            DR_CUDA(cudaEventRecord((cudaEvent_t)d->done_event, s->s_d2h));
        }
        return DR_OK;
    };
    rc = enqueue();
    // One bounded wait for the tail of each stream.  When the caller's bound runs out (or enqueueing failed half
    // way) the work already enqueued cannot be cancelled: it is waited for under a generous fixed bound, so that
    // no copy or kernel of this call still targets the caller's buffers when the call returns.
    const auto limit = std::chrono::milliseconds(d->timeout_ms ? d->timeout_ms : 60000);
    auto deadline = std::chrono::steady_clock::now() + limit;
    bool draining = rc != DR_OK;
    if (draining) deadline = std::chrono::steady_clock::now() + std::chrono::seconds(20);
    for (cudaStream_t q : {s->s_h2d, s->s_kernel, s->s_d2h}) {
        for (;;) {
            cudaError_t e = cudaStreamQuery(q);
            if (e == cudaSuccess) break;
            if (e != cudaErrorNotReady) {
                set_error("cudaStreamQuery: %s", cudaGetErrorString(e));
                return DR_ERR_CUDA;
            }
            if (std::chrono::steady_clock::now() > deadline) {
                if (draining) break;  // gave up on the drain as well: report the first error
                set_error("streamed repack wait timed out");
                rc = DR_ERR_TIMEOUT;
                draining = true;
                deadline = std::chrono::steady_clock::now() + std::chrono::seconds(20);
                continue;
            }
            std::this_thread::sleep_for(std::chrono::microseconds(50));
        }
    }
    st.elapsed_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
    if (stats) *stats = st;
    return rc;
}
