// The index object behind war_index_t (library-internal).
#pragma once
#include <stdint.h>
#include <vector>

struct war_index {
    int32_t* corpus = nullptr;   // [capacity + slack] trajectories joined by unique negative separators
    int32_t* sa = nullptr;       // [capacity]
    uint8_t* lcp = nullptr;      // [capacity + slack]
    int32_t* bucket = nullptr;   // [vocab + 1]
    int64_t M = 0;               // corpus entries in use
    int64_t capacity = 0;
    int32_t T = 0;
    int32_t vocab = 0;
    int32_t max_depth = 0;
    int device = 0;
    std::vector<int64_t> bounds{0};   // host: corpus position where each stored trajectory starts, then M
};
