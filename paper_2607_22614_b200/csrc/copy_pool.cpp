#include "copy_pool.h"

#include <algorithm>
#include <cstring>

#if defined(__x86_64__)
#include <immintrin.h>
#endif

namespace dr {
namespace {

#if defined(__x86_64__)
// Streaming copy: ordinary loads, non-temporal 32-byte stores (no read-for-ownership of the destination).
__attribute__((target("avx2"))) void stream_copy_avx2(char* dst, const char* src, uint64_t n)
{
    uint64_t head = (32 - ((uintptr_t)dst & 31)) & 31;
    if (head > n) head = n;
    memcpy(dst, src, head);
    dst += head;
    src += head;
    n -= head;
    uint64_t blocks = n / 128;
    for (uint64_t i = 0; i < blocks; ++i) {
        __m256i a = _mm256_loadu_si256((const __m256i*)(src));
        __m256i b = _mm256_loadu_si256((const __m256i*)(src + 32));
        __m256i c = _mm256_loadu_si256((const __m256i*)(src + 64));
        __m256i d = _mm256_loadu_si256((const __m256i*)(src + 96));
        _mm256_stream_si256((__m256i*)(dst), a);
        _mm256_stream_si256((__m256i*)(dst + 32), b);
        _mm256_stream_si256((__m256i*)(dst + 64), c);
        _mm256_stream_si256((__m256i*)(dst + 96), d);
        src += 128;
        dst += 128;
    }
    _mm_sfence();
    memcpy(dst, src, n - blocks * 128);
}
bool have_avx2()
{
    static const bool v = __builtin_cpu_supports("avx2");
    return v;
}
#endif

void copy_bytes(char* dst, const char* src, uint64_t n)
{
#if defined(__x86_64__)
    if (n >= (1u << 16) && have_avx2()) {
        stream_copy_avx2(dst, src, n);
        return;
    }
#endif
    memcpy(dst, src, n);
}

}  // namespace

Drainer::Drainer(unsigned n_threads)
{
    for (unsigned i = 0; i < (n_threads ? n_threads : 1); ++i) th_.emplace_back([this] { loop(); });
}

Drainer::~Drainer()
{
    {
        std::lock_guard<std::mutex> l(mu_);
        stop_ = true;
    }
    work_.notify_all();
    for (auto& t : th_) t.join();
}

void Drainer::submit(const Part* parts, unsigned n_parts, std::atomic<uint32_t>* pending)
{
    uint32_t n_tasks = 0;
    for (unsigned i = 0; i < n_parts; ++i) n_tasks += (uint32_t)((parts[i].n + kTaskBytes - 1) / kTaskBytes);
    pending->store(n_tasks, std::memory_order_release);
    if (n_tasks == 0) return;
    {
        std::lock_guard<std::mutex> l(mu_);
        for (unsigned i = 0; i < n_parts; ++i)
            for (uint64_t off = 0; off < parts[i].n; off += kTaskBytes)
                q_.push_back(Task{parts[i].dst + off, parts[i].src + off, std::min(kTaskBytes, parts[i].n - off), parts[i].cached,
                                 pending});
    }
    if (n_tasks == 1) work_.notify_one(); else work_.notify_all();
}

bool Drainer::wait_zero(const std::atomic<uint32_t>* pending, std::chrono::steady_clock::time_point deadline)
{
    if (pending->load(std::memory_order_acquire) == 0) return true;
    std::unique_lock<std::mutex> l(mu_);
    return done_.wait_until(l, deadline, [&] { return pending->load(std::memory_order_acquire) == 0; });
}

void Drainer::loop()
{
    for (;;) {
        Task t;
        {
            std::unique_lock<std::mutex> l(mu_);
            work_.wait(l, [&] { return stop_ || !q_.empty(); });
            if (q_.empty()) return;  // stop requested and nothing left to copy
            t = q_.front();
            q_.pop_front();
        }
        if (t.cached) memcpy(t.dst, t.src, t.n); else copy_bytes(t.dst, t.src, t.n);
        if (t.pending->fetch_sub(1, std::memory_order_acq_rel) == 1) {  // the chunk's last task
            std::lock_guard<std::mutex> l(mu_);                          // pairs with the waiter's predicate check
            done_.notify_all();
        }
    }
}

}  // namespace dr
