// Host-side parallel copy between the pinned staging ring and a pageable host arena.
#pragma once
#include <chrono>
#include <condition_variable>
#include <cstdint>
#include <deque>
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

// Copies finished chunks from the pinned ring to a pageable arena on a thread of its own (which in turn
// drives the CopyPool), so that the pump thread is free to issue the next device-to-host copies while a
// chunk is still being copied out.  Chunks are copied in submission order.
class Drainer {
public:
    struct Part {
        char* dst;
        const char* src;
        uint64_t n;
    };
    explicit Drainer(CopyPool* pool);
    ~Drainer();
    void submit(const Part* parts, unsigned n_parts);  // one chunk: up to one part per state buffer it touches
    uint64_t completed();                               // chunks copied out since construction
    // Blocks until `count` chunks have been copied out, or the deadline passes (returns false).
    bool wait_completed(uint64_t count, std::chrono::steady_clock::time_point deadline);

private:
    void loop();
    CopyPool* pool_;
    std::thread th_;
    std::mutex mu_;
    std::condition_variable work_, done_;
    std::deque<std::vector<Part>> q_;
    uint64_t completed_ = 0;
    bool stop_ = false;
};

}  // namespace dr
