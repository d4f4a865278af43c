// Work decomposition of the verify-attention call (library-internal).
//
// A unit = (request, kv head, row block, KV chunk).  The rows of a unit are the (slot, query head of the group)
// pairs r = slot * G + g of one kv head, cut into row blocks of at most kRowBlock rows; its chunk is a range of
// 128-key tiles.  A tiny planning kernel cuts every request into chunks so that about kTargetUnits units exist,
// orders requests longest-first and writes the unit table; the attention kernel's persistent CTAs take units in a
// fixed snake order; units of a split request leave (max, sum, unnormalised output) partials that a combine kernel merges
// in chunk order.  With few requests and one row block per kv head the plan is a contiguous split instead: the tiles
// of all (request, kv head) pairs form one sequence that is cut into equal ranges, one per CTA, so every CTA streams
// the same number of tiles whatever the lengths of the requests; a pair that crosses a cut is merged the same way.  Everything lives in the caller's workspace, so no call allocates.
#pragma once
#include <stdint.h>
#include "war.h"

constexpr int kTileKeys = 128;          // planning granularity in keys
constexpr int kRowBlock = 128;          // query rows per unit
constexpr int kTargetUnits = 148 * 8;   // aim: several units per SM of a B200 (a tuning constant of the plan, not a launch size)
constexpr int kMinChunkTiles = 8;       // never cut finer than 1024 keys
constexpr int kMaxPlanB = 4096;

struct AttnUnit {
    int req, kvh, rb, tile_begin, tile_end, n_chunks, chunk, pad;
};
struct AttnReq {
    int base_unit, n_chunks, n_tiles, n_nodes;
};

constexpr int kMaxPlanCtas = 1024;      // CTAs of the attention grid the plan can describe

struct AttnWorkspace {
    int* counters;       // [0] next unit to hand out, [1] number of units, [2] chunk size in tiles,
                         // [3] 1: contiguous split (units of CTA c are cta_first[c] .. cta_first[c+1]), 0: snake deal
    int* cta_first;      // [kMaxPlanCtas + 1]   contiguous split: first unit of every CTA
    int* pair_unit0;     // [B, Hkv]             contiguous split: unit of the first chunk of (request, kv head),
    int* pair_cta0;      // [B, Hkv]             the CTA that runs it (chunk c > 0 is the first unit of CTA cta0 + c)
    int* pair_chunks;    // [B, Hkv]             and the number of chunks
    unsigned long long* pair_count;   // [B, Hkv, row_blocks]  one-launch path: (call number << 16) | units of a split
                                      // triple that have left their partial result
    unsigned long long* pair_seen;    // [B, Hkv, row_blocks]  the same for the CTAs that share the triple's merge and have
                                      // seen all of its partials
    AttnReq* req;        // [B]
    uint64_t* anc;       // [B, N] bit a of anc[b, j]: slot a is j or an ancestor of j
    AttnUnit* units;     // [max_units]
    float* part_ml;      // [max_units, rows, 2]  running max (log2 domain) and sum
    float* part_o;       // [max_units, rows, D]  unnormalised output
    int max_units, rows, row_blocks;
    size_t bytes;
};

// Memory layout of a pool [num_pages, Hkv, page_size, D] as given by its element strides:
//   0  head-major  (page, head, token, d contiguous in this order)
//   1  token-major (page, token, head, d: the layout of engines that store a page as [block_size, heads, head_size])
//  -1  anything else
inline int war_attn_pool_layout(const int64_t* s, const war_attn_params_t* p) {
    const int64_t D = p->D, pg = p->page_size, H = p->Hkv;
    if (s[3] != 1) return -1;
    if (s[2] == D && s[1] == pg * D && s[0] == H * pg * D) return 0;
    if (s[1] == D && s[2] == H * D && s[0] == pg * H * D) return 1;
    return -1;
}

inline AttnWorkspace war_attn_workspace_layout(const war_attn_params_t* p, void* base) {
    AttnWorkspace w;
    const int G = p->Hq / p->Hkv;
    const int R = G * p->N;
    w.rows = ((R < kRowBlock ? R : kRowBlock) + 1) & ~1;        // even: a unit's (max, sum) block starts on a 16-byte boundary
    w.row_blocks = (R + kRowBlock - 1) / kRowBlock;
    w.max_units = kTargetUnits + p->B * p->Hkv * w.row_blocks;
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    size_t at = 0;
    char* b = (char*)base;
    w.counters = (int*)(b + at); at += align(64 * sizeof(int));
    w.cta_first = (int*)(b + at); at += align(sizeof(int) * (kMaxPlanCtas + 1));
    w.pair_unit0 = (int*)(b + at); at += align(sizeof(int) * (size_t)p->B * p->Hkv);
    w.pair_cta0 = (int*)(b + at); at += align(sizeof(int) * (size_t)p->B * p->Hkv);
    w.pair_chunks = (int*)(b + at); at += align(sizeof(int) * (size_t)p->B * p->Hkv);
    w.pair_count = (unsigned long long*)(b + at); at += align(sizeof(unsigned long long) * (size_t)p->B * p->Hkv * w.row_blocks);
    w.req = (AttnReq*)(b + at); at += align(sizeof(AttnReq) * (size_t)p->B);
    w.anc = (uint64_t*)(b + at); at += align(sizeof(uint64_t) * (size_t)p->B * p->N);
    w.units = (AttnUnit*)(b + at); at += align(sizeof(AttnUnit) * (size_t)w.max_units);
    w.part_ml = (float*)(b + at); at += align(sizeof(float) * 2 * (size_t)w.max_units * w.rows);
    w.part_o = (float*)(b + at); at += align(sizeof(float) * (size_t)w.max_units * w.rows * p->D);
    w.pair_seen = (unsigned long long*)(b + at); at += align(sizeof(unsigned long long) * (size_t)p->B * p->Hkv * w.row_blocks);
    w.bytes = at;
    return w;
}

// Launchers implemented per kernel family.  Both consume the same plan and leave the same partials.
war_status_t war_attn_launch_simple(const void* q, const void* k, const void* v, const int32_t* page_table,
                                    const int32_t* prefix_len, const war_attn_params_t* p, const AttnWorkspace& w,
                                    void* out, float* lse, int* status_word, cudaStream_t s);
// fused: the kernel plans for itself and merges split units itself (one launch, see war_attn_fused_plan.cuh)
war_status_t war_attn_launch_sm100(const void* q, const void* k, const void* v, const int32_t* page_table,
                                   const int32_t* prefix_len, const int32_t* num_nodes, const int32_t* parent,
                                   const war_attn_params_t* p, const AttnWorkspace& w, bool fused,
                                   void* out, float* lse, int* status_word, cudaStream_t s);
int war_attn_sm_count();                 // SMs of the current device (0 on error)
