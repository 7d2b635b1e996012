// Host-side parallel copy between the pinned staging ring and a pageable host arena.
#pragma once
#include <condition_variable>
#include <cstdint>
#include <mutex>
#include <thread>
#include <vector>

namespace dr {

// Splits one copy over a few threads (a single core cannot keep up with the host link) and writes with
// non-temporal stores where the CPU has them, so that the destination is not first read into cache.
class CopyPool {
public:
    explicit CopyPool(unsigned n_threads);
    ~CopyPool();
    void copy(void* dst, const void* src, uint64_t n);  // returns when all bytes are copied
    unsigned threads() const { return n_; }

private:
    void part(unsigned i);
    void loop(unsigned i);
    unsigned n_;
    std::vector<std::thread> th_;
    std::mutex mu_;
    std::condition_variable cv_, done_;
    uint64_t gen_ = 0;
    unsigned pending_ = 0;
    bool stop_ = false;
    char* dst_ = nullptr;
    const char* src_ = nullptr;
    uint64_t len_ = 0;
};

}  // namespace dr
