// The index object behind war_index_t (library-internal).
#pragma once
#include <stdint.h>
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

struct war_index {
    int32_t* corpus = nullptr;   // [capacity + slack] trajectories joined by unique negative separators
    war_index_arrays set[2];
    int cur = 0;                 // published set; guarded by `lock` together with the pointers handed to queries
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
    void publish() { std::lock_guard<std::mutex> g(lock); cur ^= 1; }
};
