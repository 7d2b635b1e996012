// Host-side parallel copies between the pinned staging ring and a pageable host arena.
#pragma once
#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstdint>
#include <deque>
#include <mutex>
#include <thread>
#include <vector>

namespace dr {

// Copies finished chunks from the pinned ring to a pageable arena on worker threads of its own, so that the pump
// thread is free to issue the next device-to-host copies while chunks are still being copied out.  A chunk's parts
// are cut into tasks of at most kTaskBytes that any worker may take: a large chunk is spread over all workers, and
// several small chunks are copied side by side (small chunks, copied right behind the DMA that delivered them, can
// be read from the last-level cache instead of from DRAM on hosts whose I/O writes allocate there).
class Drainer {
public:
    struct Part {
        char* dst;
        const char* src;
        uint64_t n;
        bool cached = false;  // ordinary stores (the destination is about to be read by the device from the cache)
    };
    static constexpr uint64_t kTaskBytes = 1ull << 20;
    explicit Drainer(unsigned n_threads);
    ~Drainer();
    // Queue the parts of one chunk.  *pending receives the number of tasks and is counted down as they finish.
    void submit(const Part* parts, unsigned n_parts, std::atomic<uint32_t>* pending);
    // Blocks until *pending is zero, or the deadline passes (returns false).
    bool wait_zero(const std::atomic<uint32_t>* pending, std::chrono::steady_clock::time_point deadline);

private:
    struct Task {
        char* dst;
        const char* src;
        uint64_t n;
        bool cached;
        std::atomic<uint32_t>* pending;
    };
    void loop();
    std::vector<std::thread> th_;
    std::mutex mu_;
    std::condition_variable work_, done_;
    std::deque<Task> q_;
    bool stop_ = false;
};

}  // namespace dr
