// The index object behind war_index_t (library-internal).
#pragma once
#include <stdint.h>
#include <cuda_runtime.h>
#include <mutex>
#include <vector>

// The arrays a query reads.  There are two sets: queries read the published one, every update writes the other one
// and publishes it when it is complete, so a query that was enqueued before an update returned keeps reading a
// complete index.  The corpus is shared by both sets: an append only writes behind what the old set refers to.
struct war_index_arrays {
    int32_t* sa = nullptr;       // [capacity]
    uint8_t* lcp = nullptr;      // [capacity + slack]
    int32_t* bucket = nullptr;   // [vocab + 1]
    int32_t* memo = nullptr;     // [kMemoEntries * kMemoInts] expansions of large nodes, filled by the draft kernel
};

// Memo of node expansions (library-internal cache, part of a set: it describes that set's suffix array).  The draft
// kernel spends most of a slow request in nodes with many occurrences (one- and two-token strings of frequent
// tokens), and those nodes are the same for every request and step until the index changes.  An entry holds the
// k best continuations of one node: key (lo + 1, depth, k), state, n, then count / start / token per continuation.
constexpr int kMemoEntries = 1 << 16;
constexpr int kMemoInts = 32;             // 128 bytes per entry

// What a draft kernel needs of the index, readable on the device: both array sets (their addresses never change after
// the build) and the number of the published one.  Kernels take the published set through this view when they START,
// not when they are enqueued, so a launch captured in a CUDA graph follows the index through later updates.
struct war_index_view {
    war_index_arrays set[2];
    unsigned int cur;            // written in stream order by every publication
};

struct war_index {
    int32_t* corpus = nullptr;   // [capacity + slack] trajectories joined by unique negative separators
    war_index_arrays set[2];
    war_index_view* d_view = nullptr;   // device copy of (set, cur)
    // stream-ordered append: pinned staging memory for a batch's trajectory bounds, and the event after which it is free again
    static constexpr size_t kStageEntries = 1 << 16;
    int64_t* h_stage = nullptr;
    cudaEvent_t stage_free = nullptr;
    int cur = 0;                 // published set (host copy); guarded by `lock` together with the pointers handed to queries
    std::mutex lock;
    int64_t M = 0;               // corpus entries in use
    int64_t capacity = 0;
    int32_t T = 0;
    int32_t vocab = 0;
    int32_t max_depth = 0;
    int device = 0;
    std::vector<int64_t> bounds{0};   // host: corpus position where each stored trajectory starts, then M

    war_index_arrays published() { std::lock_guard<std::mutex> g(lock); return set[cur]; }
    war_index_arrays& shadow() { return set[cur ^ 1]; }                  // only the (single) updater touches it
    // Publication: the device view first (on the updater's stream, behind everything that built the set; the caller
    // synchronises that stream before it reports success), then the host copy.
    cudaError_t publish(cudaStream_t s) {
        const unsigned int next = (unsigned int)(cur ^ 1);
        cudaError_t e = cudaMemcpyAsync(&d_view->cur, &next, sizeof(next), cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return e;
        std::lock_guard<std::mutex> g(lock);
        cur ^= 1;
        return cudaSuccess;
    }
};
