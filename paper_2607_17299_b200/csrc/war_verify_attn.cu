// Verify attention: argument checks, the planning kernel, the split-KV combine kernel and the plain CUDA-core
// attention kernel (kept as the A/B reference of the tensor-core kernel in war_verify_attn_sm100.cu).
#include <cuda_bf16.h>
#include <math_constants.h>
#include "war_common.cuh"
#include "war_attn_plan.cuh"
#include "war_attn_fused_plan.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ------------------------------------------------------------------------------------------------
// plan: one CTA
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint64_t shfl64(uint64_t v, int src) {
    const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)v, src);
    const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(v >> 32), src);
    return ((uint64_t)hi << 32) | lo;
}

// The contiguous split of the plan (see attn_plan_kernel): units of every CTA, per-pair records for the merge.
// Kept out of line so that calls which do not use it run through the same code as before.  All positions are 32-bit
// (the caller checked that the sequence has fewer than 2^31 tiles) and the cuts are worked out once, one 64-bit division
// per CTA in parallel: everything after that is additions, comparisons and 32-bit divisions.
__device__ __noinline__ void plan_contiguous(const int* s_tiles, const uint8_t* s_n, int* s_start, int* s_cnt, int* s_cut, int B,
                                             int Hkv, int n_ctas, int rows_max, int pairs, AttnWorkspace w) {
    __shared__ int s_live_before[65], s_weight[64];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (warp == 0) {                                             // first tile of every request's pairs in the sequence
        const int q0 = 2 * lane, q1 = 2 * lane + 1;              // two requests per lane: B <= 64
        const int l0 = q0 < B && s_n[q0] > 0 && s_tiles[q0] > 0, l1 = q1 < B && s_n[q1] > 0 && s_tiles[q1] > 0;
        const int m0 = l0 ? s_tiles[q0] * Hkv : 0, m1 = l1 ? s_tiles[q1] * Hkv : 0;
        int incl = m0 + m1, live = l0 + l1;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o), z = __shfl_up_sync(0xffffffffu, live, o);
            if (lane >= o) { incl += y; live += z; }
        }
        s_start[q0] = incl - m0 - m1;
        s_start[q1] = incl - m1;
        s_live_before[q0] = live - l0 - l1;
        s_live_before[q1] = live - l1;
        s_weight[q0] = l0; s_weight[q1] = l1;
        if (lane == 31) s_start[64] = incl;
    }
    __syncthreads();
    const int t_all = s_start[64];
    const int n_used = min(n_ctas, max(1, t_all / 4));           // at least four tiles per CTA
    // the cuts of the one-launch path (a pair costs its tiles plus the cost of a unit)
    const int unit_cost = fused_plan::contiguous_unit_cost(rows_max);
    for (int c = tid; c <= n_used; c += 1024)
        s_cut[c] = fused_plan::contiguous_cut(c, n_used, t_all, pairs, unit_cost, s_tiles, s_weight, s_start, s_live_before, B, Hkv);
    __syncthreads();
    auto req_of = [&](int x) -> int {                            // request whose pairs hold tile x of the sequence
        int r = 0;
        for (int q = 1; q < B; ++q) if (s_start[q] <= x && s_n[q] > 0 && s_tiles[q] > 0) r = q;
        return r;
    };
    auto cta_of = [&](int x) -> int {                            // the CTA whose (non-empty) range holds tile x
        int c = min(n_used - 1, x / max(1, t_all / n_used));       // a guess, then steps along the cuts
        while (c + 1 < n_used && s_cut[c + 1] <= x) ++c;
        while (c > 0 && s_cut[c] > x) --c;
        return c;
    };
    // the units of every CTA, one thread per CTA: first how many (one per pair that overlaps its range), then, after
    // a scan, the units themselves
    int r0 = 0, r1 = -1, h_first = 0, h_last = 0, lo = 0, hi = 0;
    if (tid < n_used) {
        lo = s_cut[tid]; hi = s_cut[tid + 1];
        if (hi > lo) {
            r0 = req_of(lo); r1 = req_of(hi - 1);
            h_first = (lo - s_start[r0]) / s_tiles[r0]; h_last = (hi - 1 - s_start[r1]) / s_tiles[r1];
        }
    }
    for (int c = tid; c < n_used; c += 1024) {                   // (n_used <= 1024: one pass)
        int cnt = 0;
        for (int r = r0; r <= r1; ++r) {
            if (s_n[r] <= 0 || s_tiles[r] <= 0) continue;
            cnt += (r == r1 ? h_last : Hkv - 1) - (r == r0 ? h_first : 0) + 1;
        }
        s_cnt[c] = cnt;
    }
    __syncthreads();
    if (warp == 0) {                                             // exclusive scan over the CTAs: a segment per lane
        const int per = (n_used + 31) / 32, c0 = lane * per, c1 = min(n_used, c0 + per);
        int sum = 0;
        for (int c = c0; c < c1; ++c) sum += s_cnt[c];
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        int run = incl - sum;
        for (int c = c0; c < c1; ++c) { const int x = s_cnt[c]; s_cnt[c] = run; run += x; }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (lane == 0) { s_cnt[n_used] = total; w.counters[0] = 0; w.counters[1] = total; w.counters[2] = 0; w.counters[3] = 1; }
    }
    __syncthreads();
    for (int c = tid; c <= n_ctas; c += 1024) w.cta_first[c] = s_cnt[min(c, n_used)];
    for (int i = tid; i < B; i += 1024) {
        AttnReq rq;
        rq.base_unit = -1; rq.n_chunks = 2; rq.n_tiles = s_tiles[i]; rq.n_nodes = s_n[i];  // -1: contiguous split, see pair_chunks
        w.req[i] = rq;
    }
    for (int i = tid; i < B * Hkv; i += 1024)
        if (s_n[i / Hkv] <= 0 || s_tiles[i / Hkv] <= 0) w.pair_chunks[i] = 0;
    if (tid < n_used && hi > lo) {
        const int c = tid;
        int u = s_cnt[c];
        for (int r = r0; r <= r1; ++r) {
            const int t = s_tiles[r];
            if (s_n[r] <= 0 || t <= 0) continue;
            const int h0 = r == r0 ? h_first : 0, h1 = r == r1 ? h_last : Hkv - 1;
            for (int h = h0; h <= h1; ++h, ++u) {
                const int ps = s_start[r] + h * t;                                       // the pair's first tile
                // a pair that starts in this range and ends in it is whole; otherwise look the two ends up
                const int c0 = ps >= lo ? c : cta_of(ps), c1 = ps + t <= hi ? c : cta_of(ps + t - 1);
                AttnUnit x;
                x.req = r; x.kvh = h; x.rb = 0;
                x.tile_begin = max(lo, ps) - ps; x.tile_end = min(hi, ps + t) - ps;
                x.n_chunks = c1 - c0 + 1; x.chunk = c - c0; x.pad = 0;
                w.units[u] = x;
                if (c == c0) { w.pair_unit0[r * Hkv + h] = u; w.pair_cta0[r * Hkv + h] = c0; w.pair_chunks[r * Hkv + h] = c1 - c0 + 1; }
            }
        }
    }
}

constexpr int kSearchMaxB = 64;           // up to this many requests the chunk length is searched (see below)

__global__ void __launch_bounds__(1024)
attn_plan_kernel(const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ num_nodes,
                 const int32_t* __restrict__ parent, int B, int N, int Hkv, int G, int page_size, int max_pages, int n_ctas,
                 AttnWorkspace w, int* status_word) {
    constexpr int kPer = kMaxPlanB / 1024;    // requests per thread in the per-request phases
    __shared__ int s_tiles[kMaxPlanB];
    __shared__ int s_units[kMaxPlanB];        // units per request, indexed by sorted position; then exclusive scan
    __shared__ uint16_t s_order[kMaxPlanB];   // request at each sorted position
    __shared__ uint8_t s_n[kMaxPlanB];        // validated slot count
    __shared__ int s_red[32];
    __shared__ long long s_sum[32], s_sum2[32];
    __shared__ int s_chunk_tiles, s_total, s_one_wave, s_cstar;
    __shared__ long long s_tot;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- per request, one warp: validate, ancestor masks by pointer jumping, tile count ----
    // Lane l holds slots l and l + 32.  After round r a slot's mask covers its 2^r nearest ancestors-or-self and its
    // pointer is the 2^r-th ancestor (the root points at itself), so 6 rounds cover any tree of 64 slots.
    // The parent row is requested together with the slot count (all N entries exist; the ones past n are ignored), and
    // the next request's while this one is worked on: the warp waits for one memory latency in all, not two per request.
    const int j0 = lane, j1 = lane + 32;
    int nx_q0 = 0, nx_q1 = 0, nx_n = 0, nx_pl = 0;
    if (warp < B) {
        const int32_t* prow = parent + (size_t)warp * N;
        nx_q0 = j0 < N ? prow[j0] : 0; nx_q1 = j1 < N ? prow[j1] : 0;
        nx_n = num_nodes[warp]; nx_pl = prefix_len[warp];
    }
    for (int i = warp; i < B; i += 32) {
        const int q0 = nx_q0, q1 = nx_q1;
        int n = nx_n;
        const int pl = nx_pl;
        if (i + 32 < B) {
            const int32_t* prow = parent + (size_t)(i + 32) * N;
            nx_q0 = j0 < N ? prow[j0] : 0; nx_q1 = j1 < N ? prow[j1] : 0;
            nx_n = num_nodes[i + 32]; nx_pl = prefix_len[i + 32];
        }
        bool bad = n < 0 || n > N || pl < 0;
        if (!bad && n > 0) {
            int p0 = (j0 > 0 && j0 < n) ? q0 : 0;
            int p1 = (j1 < n) ? q1 : 0;
            const bool bad_l = (j0 > 0 && j0 < n && (p0 < 0 || p0 >= j0)) || (j1 < n && (p1 < 0 || p1 >= j1));
            bad = __any_sync(0xffffffffu, bad_l);
            if (!bad) {
                uint64_t a0 = 1ull << j0, a1 = 1ull << j1;
                if (n <= 32) {
#pragma unroll
                    for (int r = 0; r < 5; ++r) {
                        const uint64_t b = shfl64(a0, p0);
                        const int q = __shfl_sync(0xffffffffu, p0, p0);
                        a0 |= b; p0 = q;
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < 6; ++r) {
                        const uint64_t b00 = shfl64(a0, p0 & 31), b01 = shfl64(a1, p0 & 31);
                        const uint64_t b10 = shfl64(a0, p1 & 31), b11 = shfl64(a1, p1 & 31);
                        const int q00 = __shfl_sync(0xffffffffu, p0, p0 & 31), q01 = __shfl_sync(0xffffffffu, p1, p0 & 31);
                        const int q10 = __shfl_sync(0xffffffffu, p0, p1 & 31), q11 = __shfl_sync(0xffffffffu, p1, p1 & 31);
                        a0 |= p0 >= 32 ? b01 : b00;
                        a1 |= p1 >= 32 ? b11 : b10;
                        p0 = p0 >= 32 ? q01 : q00;
                        p1 = p1 >= 32 ? q11 : q10;
                    }
                }
                if (j0 < n) w.anc[(size_t)i * N + j0] = a0;
                if (j1 < n) w.anc[(size_t)i * N + j1] = a1;
            }
        }
        if (lane == 0) {
            if (bad) { war_set_device_status(status_word, WAR_ERR_BAD_TREE); n = 0; }
            int tiles = 0;
            if (n > 0) {
                const long long L = (long long)pl + n;
                if ((L + page_size - 1) / page_size > max_pages) { war_set_device_status(status_word, WAR_ERR_BAD_PAGE); n = 0; }
                else tiles = (int)((L + kTileKeys - 1) / kTileKeys);
            }
            s_tiles[i] = tiles;
            s_n[i] = (uint8_t)n;
        }
    }
    __syncthreads();

    // ---- few requests, one row block each: contiguous split ----
    // The tiles of all (request, kv head) pairs, request after request and head after head, form one sequence of
    // T_all tiles; CTA c takes the range [c * T_all / n_used, (c + 1) * T_all / n_used).  A pair that crosses a cut is
    // split there: its first chunk is somewhere in a CTA's list, every further chunk is the first unit of the next CTA.
    // Every CTA streams the same number of tiles (within one) whatever the requests' lengths are.  When it pays:
    // fused_plan::contiguous_split_pays (the one-launch path takes the same decision in every CTA).
    if (B <= 64 && n_ctas <= kMaxPlanCtas) {
        // every warp works the rule out for itself (two requests per lane): no barrier on the way of the calls that do not use it
        int n_mx = 0, prs = 0, t_mx = 0, t_sm = 0;
        for (int q = lane; q < B; q += 32) {
            const int n = s_n[q], t = s_tiles[q];
            n_mx = max(n_mx, n);
            if (n > 0 && t > 0) { prs += Hkv; t_mx = max(t_mx, t); t_sm += t; }
        }
        const int rows_max = G * __reduce_max_sync(0xffffffffu, n_mx);
        const int pairs = __reduce_add_sync(0xffffffffu, prs);
        const int t_max = __reduce_max_sync(0xffffffffu, t_mx);
        const int t_sum = __reduce_add_sync(0xffffffffu, t_sm);               // < 2^31: at most 64 requests of < 2^24 tiles
        const long long t_all = (long long)t_sum * Hkv;
        (void)t_max;
        if (fused_plan::contiguous_split_pays(rows_max, t_all, n_ctas)) {
            __shared__ int s_start[65];
            plan_contiguous(s_tiles, s_n, s_start, s_units, s_units + kMaxPlanCtas + 8, B, Hkv, n_ctas, rows_max, pairs, w);   // (the snake deal's s_units is free here)
            return;
        }
    }

    // ---- per request, one thread: weights, order, chunk counts ----
    int r_n[kPer], r_tiles[kPer], r_rbs[kPer], r_pos[kPer], r_nc[kPer];
    long long my_tiles = 0;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int i = tid + k * 1024;
        r_n[k] = 0; r_tiles[k] = 0; r_rbs[k] = 0; r_pos[k] = 0; r_nc[k] = 0;
        if (i >= B) continue;
        r_n[k] = s_n[i]; r_tiles[k] = s_tiles[i];
        r_rbs[k] = r_n[k] > 0 ? (G * r_n[k] + kRowBlock - 1) / kRowBlock : 0;
        my_tiles += (long long)r_tiles[k] * r_rbs[k];
    }
    // block sum of tiles (weighted by row blocks and kv heads)
    for (int o = 16; o > 0; o >>= 1) my_tiles += __shfl_xor_sync(0xffffffffu, my_tiles, o);
    if (lane == 0) s_sum[warp] = my_tiles;
    __syncthreads();
    if (tid == 0) {
        long long tot = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += s_sum[i];
        tot *= Hkv;
        long long ct = (tot + kTargetUnits - 1) / kTargetUnits;
        if (ct < kMinChunkTiles) ct = kMinChunkTiles;
        s_chunk_tiles = (int)ct;
        s_tot = tot;
        s_one_wave = 0;
        w.counters[0] = 0;
        w.counters[2] = (int)ct;
        w.counters[3] = 0;
    }
    __syncthreads();
    const int chunk_tiles = s_chunk_tiles;
    // Little work (few requests): the default chunk (about kTargetUnits units) would cut every request into short
    // units, and a unit costs about six tiles on top of its own (pipeline fill, Q load, partials written and merged;
    // calibrated on 2 to 32 requests).
    // Up to 64 requests, the block therefore looks for the chunk length c that minimises the estimated time in tiles
    //     ceil(units(c) / CTAs) * (c + 6),     units(c) = sum over (request, kv head, row block) of ceil(tiles / c),
    // over c from the default up to the longest request (fused_plan::chunk_search, the routine the one-launch path
    // runs in every CTA, so both paths cut the requests the same way).  This covers "one unit per CTA" (units(c) <=
    // CTAs: one pipeline fill and one epilogue per CTA) as well as a few long units per CTA, and with a dozen requests
    // of very different lengths it avoids leaving most CTAs idle while the longest request finishes.  Equal estimates take the longer
    // chunk (fewer partials).  More requests (only with very few kv heads can that be little work): shares of the grid
    // in proportion to the tiles, rounded down, if that fits the grid and its longest unit beats the default plan.
    const long long tot_all = s_tot;
    if (B <= kSearchMaxB) {
        __shared__ int s_keys[64];
        __shared__ int s_weight[kSearchMaxB];
        int t_mine = 0;
        for (int q = lane; q < B; q += 32) if (s_n[q] > 0) t_mine = max(t_mine, s_tiles[q]);
        const int t_max = __reduce_max_sync(0xffffffffu, t_mine);
        if (tid < kSearchMaxB) s_weight[tid] = tid < B && s_n[tid] > 0 && s_tiles[tid] > 0 ? Hkv * ((G * s_n[tid] + kRowBlock - 1) / kRowBlock) : 0;
        if (tid >= B && tid < kSearchMaxB) s_tiles[tid] = 0;
        __syncthreads();
        const int best_c = fused_plan::chunk_search<kFusedThreads>(s_tiles, s_weight, B, max(fused_plan::chunk_floor(t_max), chunk_tiles), t_max, n_ctas, s_keys);
        if (tid == 0) s_cstar = best_c;
        __syncthreads();
    }
    const int c_best = s_cstar;
    auto chunks_one_wave = [&](int t) -> int {
        if (t <= 0) return 0;
        long long nc = tot_all > 0 ? (long long)t * n_ctas / tot_all : 1;        // tot_all: the tiles of all such triples
        const int cap = max(1, t / 4);                                           // a chunk keeps at least four tiles
        return (int)max(1ll, min(nc, (long long)cap));
    };
    if (B > kSearchMaxB) {
        long long mine = 0, mine_chunked = 0;
        int longest = 0;
#pragma unroll
        for (int k = 0; k < kPer; ++k) {
            const int nc = chunks_one_wave(r_tiles[k]);
            mine += (long long)nc * Hkv * r_rbs[k];
            if (nc > 0 && r_rbs[k] > 0) longest = max(longest, (r_tiles[k] + nc - 1) / nc);
            mine_chunked += (long long)((r_tiles[k] + chunk_tiles - 1) / chunk_tiles) * Hkv * r_rbs[k];
        }
        for (int o = 16; o > 0; o >>= 1) {
            mine += __shfl_xor_sync(0xffffffffu, mine, o);
            mine_chunked += __shfl_xor_sync(0xffffffffu, mine_chunked, o);
            longest = max(longest, __shfl_xor_sync(0xffffffffu, longest, o));
        }
        __syncthreads();                                                   // s_sum is read above
        if (lane == 0) { s_sum[warp] = mine; s_sum2[warp] = mine_chunked; s_red[warp] = longest; }
        __syncthreads();
        if (tid == 0) {
            long long units = 0, units_chunked = 0;
            int lg = 0;
            for (int i = 0; i < (int)(blockDim.x >> 5); ++i) { units += s_sum[i]; units_chunked += s_sum2[i]; lg = max(lg, s_red[i]); }
            const long long t_one = lg + 2, t_chunked = ((units_chunked + n_ctas - 1) / n_ctas) * (chunk_tiles + 2);
            s_one_wave = units <= n_ctas && t_one <= t_chunked;
        }
        __syncthreads();
    }
    const bool one_wave = s_one_wave != 0;
    auto chunks_of = [&](int t) -> int {
        if (t <= 0) return 0;
        if (B <= kSearchMaxB) return (t + c_best - 1) / c_best;
        return one_wave ? chunks_one_wave(t) : (t + chunk_tiles - 1) / chunk_tiles;
    };
    // longest-first order: position = number of requests that rank before this one
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int i = tid + k * 1024;
        if (i >= B) continue;
        const int t = r_tiles[k];
        int pos = 0;
        for (int q = 0; q < B; ++q) {
            const int tq = s_tiles[q];
            pos += (tq > t) || (tq == t && q < i);
        }
        r_pos[k] = pos;
        r_nc[k] = chunks_of(t);
        s_units[pos] = r_nc[k] * Hkv * r_rbs[k];
        s_order[pos] = (uint16_t)i;
    }
    __syncthreads();
    // exclusive scan of s_units: per-thread serial segments + warp scans
    {
        const int per = (B + blockDim.x - 1) / blockDim.x;
        const int b0 = tid * per, b1 = min(B, b0 + per);
        int sum = 0;
        for (int q = b0; q < b1; ++q) sum += s_units[q];
        int incl = sum;
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        if (lane == 31) s_red[warp] = incl;
        __syncthreads();
        if (tid < 32) {
            int x = s_red[tid], xi = x;
            for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, xi, o); if (tid >= o) xi += y; }
            s_red[tid] = xi - x;
            if (tid == 31) { w.counters[1] = xi; s_total = xi; }     // total number of units
        }
        __syncthreads();
        int run = s_red[warp] + incl - sum;
        for (int q = b0; q < b1; ++q) { const int u = s_units[q]; s_units[q] = run; run += u; }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int i = tid + k * 1024;
        if (i >= B) continue;
        AttnReq rq;
        rq.base_unit = s_units[r_pos[k]]; rq.n_chunks = r_nc[k]; rq.n_tiles = r_tiles[k]; rq.n_nodes = r_n[k];
        w.req[i] = rq;
    }
    // ---- unit table, one thread per unit: per request, chunks balanced to within one tile, order (chunk, kv head,
    // row block).  Requests with units come first in the order and their offsets increase strictly, so the request of
    // unit u is the last position whose offset is <= u.
    const int total = s_total;
    for (int u = tid; u < total; u += 1024) {
        int lo = 0, hi = B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (s_units[mid] <= u) lo = mid; else hi = mid - 1;
        }
        const int i = s_order[lo];
        const int t = s_tiles[i], n = s_n[i];
        const int rbs = (G * n + kRowBlock - 1) / kRowBlock;
        const int nc = chunks_of(t);
        const int local = u - s_units[lo];
        const int c = local / (Hkv * rbs), rem = local % (Hkv * rbs);
        AttnUnit x;
        x.req = i; x.kvh = rem / rbs; x.rb = rem % rbs;
        if (t < 32768 && nc < 32768) {                              // 32-bit arithmetic is enough (and several times faster)
            x.tile_begin = (int)((unsigned)t * (unsigned)c / (unsigned)nc); x.tile_end = (int)((unsigned)t * (unsigned)(c + 1) / (unsigned)nc);
        } else {
            x.tile_begin = (int)((long long)t * c / nc); x.tile_end = (int)((long long)t * (c + 1) / nc);
        }
        x.n_chunks = nc; x.chunk = c; x.pad = 0;
        w.units[u] = x;
    }
}

// ------------------------------------------------------------------------------------------------
// combine: merges the partials of split requests in chunk order (deterministic)
// ------------------------------------------------------------------------------------------------
constexpr int kCombineWarps = 4;

// One warp per output row: lanes first reduce the chunk maxima, then stream the chunks' partial rows (float4 per
// lane, all loads independent) and accumulate in chunk order.
__global__ void __launch_bounds__(kCombineWarps * 32)
attn_combine_kernel(AttnWorkspace w, int N, int Hq, int Hkv, int G, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int i = blockIdx.x / Hkv, kvh = blockIdx.x % Hkv;
    const AttnReq rq = w.req[i];
    if (rq.n_chunks <= 1 || rq.n_nodes <= 0) return;
    const int R = G * rq.n_nodes;
    const int rbs = (R + kRowBlock - 1) / kRowBlock;
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.y * kCombineWarps + (threadIdx.x >> 5);
    if (r >= R) return;
    const int rb = r / kRowBlock, rr = r % kRowBlock;
    const int u0 = rq.base_unit + kvh * rbs + rb, ustep = Hkv * rbs;       // snake deal: unit of chunk c = u0 + c * ustep
    const bool contiguous = rq.base_unit < 0;                             // (the flag rides in the record that is read anyway)
    const int pair = i * Hkv + kvh;
    const int n_chunks = contiguous ? w.pair_chunks[pair] : rq.n_chunks;
    if (n_chunks <= 1) return;                                             // the attention kernel wrote the result itself
    const int first_unit = contiguous ? w.pair_unit0[pair] : u0, first_cta = contiguous ? w.pair_cta0[pair] : 0;
    auto unit_of = [&](int c) -> int {
        if (!contiguous) return u0 + c * ustep;
        return c == 0 ? first_unit : w.cta_first[first_cta + c];           // a later chunk opens the next CTA's list
    };
    const int my_unit = contiguous && lane < n_chunks ? unit_of(lane) : 0;   // contiguous split: the first 32 chunks' units, one per lane
    float M = -CUDART_INF_F;
    for (int c = lane; c < n_chunks; c += 32)
        M = fmaxf(M, w.part_ml[((size_t)(contiguous && c < 32 ? my_unit : unit_of(c)) * w.rows + rr) * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = 0; c < n_chunks; ++c) {
        const int uc = !contiguous ? u0 + c * ustep : c < 32 ? __shfl_sync(0xffffffffu, my_unit, c) : unit_of(c);   // (warp-uniform)
        const size_t base = (size_t)uc * w.rows + rr;
        const float2 ml = *reinterpret_cast<const float2*>(w.part_ml + base * 2);
        const float4 o = *reinterpret_cast<const float4*>(w.part_o + base * 128 + lane * 4);
        const float sc = ml.x == -CUDART_INF_F ? 0.f : exp2f(ml.x - M);
        l = fmaf(ml.y, sc, l);
        acc.x = fmaf(o.x, sc, acc.x); acc.y = fmaf(o.y, sc, acc.y); acc.z = fmaf(o.z, sc, acc.z); acc.w = fmaf(o.w, sc, acc.w);
    }
    const float inv = 1.f / l;
    const int j = r / G, g = r % G;
    const size_t row = ((size_t)i * N + j) * Hq + kvh * G + g;
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), h1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
    uint2 packed;
    packed.x = *reinterpret_cast<const uint32_t*>(&h0);
    packed.y = *reinterpret_cast<const uint32_t*>(&h1);
    *reinterpret_cast<uint2*>(out + row * 128 + lane * 4) = packed;
    if (lse && lane == 0) lse[row] = (M + log2f(l)) * kLn2;
}

// ------------------------------------------------------------------------------------------------
// plain attention kernel: one thread per query row, K/V tiles staged in shared memory
// ------------------------------------------------------------------------------------------------
constexpr int kSimpleTile = 32;
constexpr int kSimpleSub = 16;

__global__ void __launch_bounds__(128)
attn_simple_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ kpool,
                   const __nv_bfloat16* __restrict__ vpool, const int32_t* __restrict__ page_table,
                   const int32_t* __restrict__ prefix_len, int N, int Hq, int Hkv, int G, int page_size, int max_pages,
                   long long s_page, long long s_head, long long s_tok, long long num_pages, float scale_log2, AttnWorkspace w, __nv_bfloat16* __restrict__ out,
                   float* __restrict__ lse, int* status_word) {
    __shared__ __align__(16) __nv_bfloat16 sK[kSimpleTile][128];
    __shared__ __align__(16) __nv_bfloat16 sV[kSimpleTile][128];
    __shared__ int s_unit;
    const int tid = threadIdx.x;
    while (true) {
        __syncthreads();
        if (tid == 0) s_unit = atomicAdd(&w.counters[0], 1);
        __syncthreads();
        const int u = s_unit;
        if (u >= w.counters[1]) break;
        const AttnUnit un = w.units[u];
        const int i = un.req;
        const int n = w.req[i].n_nodes;
        const int R = G * n;
        const int pl = prefix_len[i];
        const int L = pl + n;
        const int r = un.rb * kRowBlock + tid;
        const bool active = r < R;
        const int j = active ? r / G : 0, g = active ? r % G : 0;
        const size_t qrow = ((size_t)i * N + j) * Hq + un.kvh * G + g;
        __nv_bfloat162 qv[64];
        {
            const uint4* src = reinterpret_cast<const uint4*>(q + qrow * 128);
#pragma unroll
            for (int c = 0; c < 16; ++c) {
                uint4 x = active ? src[c] : make_uint4(0, 0, 0, 0);
                qv[4 * c + 0] = *reinterpret_cast<__nv_bfloat162*>(&x.x);
                qv[4 * c + 1] = *reinterpret_cast<__nv_bfloat162*>(&x.y);
                qv[4 * c + 2] = *reinterpret_cast<__nv_bfloat162*>(&x.z);
                qv[4 * c + 3] = *reinterpret_cast<__nv_bfloat162*>(&x.w);
            }
        }
        const uint64_t anc = active ? w.anc[(size_t)i * N + j] : 0ull;
        float m = -CUDART_INF_F, l = 0.f;
        float acc[128];
#pragma unroll
        for (int d = 0; d < 128; ++d) acc[d] = 0.f;
        const int k_begin = un.tile_begin * kTileKeys;
        const int k_end = min(un.tile_end * kTileKeys, L);
        for (int kt = k_begin; kt < k_end; kt += kSimpleTile) {
            __syncthreads();
            // stage 32 keys x 256 B of K and of V: 16-byte pieces, 16 per row
            for (int x = tid; x < kSimpleTile * 16 * 2; x += 128) {
                const int which = x / (kSimpleTile * 16), y = x % (kSimpleTile * 16);
                const int row = y / 16, piece = y % 16;
                const int pos = kt + row;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (pos < k_end) {
                    long long page = page_table[(size_t)i * max_pages + pos / page_size];
                    if (page < 0 || page >= num_pages) { war_set_device_status(status_word, WAR_ERR_BAD_PAGE); page = 0; }
                    const __nv_bfloat16* pool = which ? vpool : kpool;
                    const size_t off = (size_t)(page * s_page + un.kvh * s_head + (pos % page_size) * s_tok) + piece * 8;
                    val = *reinterpret_cast<const uint4*>(pool + off);
                }
                *reinterpret_cast<uint4*>(&(which ? sV : sK)[row][piece * 8]) = val;
            }
            __syncthreads();
            if (!active) continue;
            for (int sub = 0; sub < kSimpleTile; sub += kSimpleSub) {
                float s[kSimpleSub];
                float tmax = -CUDART_INF_F;
#pragma unroll
                for (int kk = 0; kk < kSimpleSub; ++kk) {
                    const int pos = kt + sub + kk;
                    const __nv_bfloat162* krow = reinterpret_cast<const __nv_bfloat162*>(&sK[sub + kk][0]);
                    float a = 0.f;
#pragma unroll
                    for (int d = 0; d < 64; ++d) {
                        const float2 kf = __bfloat1622float2(krow[d]);
                        const float2 qf = __bfloat1622float2(qv[d]);
                        a = fmaf(qf.x, kf.x, a);
                        a = fmaf(qf.y, kf.y, a);
                    }
                    const bool vis = pos < pl || (pos < k_end && ((anc >> (pos - pl)) & 1ull));
                    s[kk] = vis ? a * scale_log2 : -CUDART_INF_F;
                    tmax = fmaxf(tmax, s[kk]);
                }
                if (tmax == -CUDART_INF_F) continue;
                const float m_new = fmaxf(m, tmax);
                const float corr = exp2f(m - m_new);          // m = -inf on the first visible key: corr = 0
                l *= corr;
#pragma unroll
                for (int d = 0; d < 128; ++d) acc[d] *= corr;
                m = m_new;
#pragma unroll
                for (int kk = 0; kk < kSimpleSub; ++kk) {
                    const float p = exp2f(s[kk] - m);          // masked: exp2(-inf) = 0
                    l += p;
                    const __nv_bfloat162* vrow = reinterpret_cast<const __nv_bfloat162*>(&sV[sub + kk][0]);
#pragma unroll
                    for (int d = 0; d < 64; ++d) {
                        const float2 vf = __bfloat1622float2(vrow[d]);
                        acc[2 * d] = fmaf(p, vf.x, acc[2 * d]);
                        acc[2 * d + 1] = fmaf(p, vf.y, acc[2 * d + 1]);
                    }
                }
            }
        }
        if (active) {
            if (un.n_chunks == 1) {
                const float inv = 1.f / l;
                __nv_bfloat162* dst = reinterpret_cast<__nv_bfloat162*>(out + qrow * 128);
#pragma unroll
                for (int d = 0; d < 64; ++d) dst[d] = __floats2bfloat162_rn(acc[2 * d] * inv, acc[2 * d + 1] * inv);
                if (lse) lse[qrow] = (m + log2f(l)) * kLn2;
            } else {
                float* po = w.part_o + ((size_t)u * w.rows + tid) * 128;
#pragma unroll
                for (int d = 0; d < 128; ++d) po[d] = acc[d];
                w.part_ml[((size_t)u * w.rows + tid) * 2] = m;
                w.part_ml[((size_t)u * w.rows + tid) * 2 + 1] = l;
            }
        }
    }
}

war_status_t check_params(const war_attn_params_t* p) {
    if (!p) return WAR_ERR_INVALID_ARG;
    if (p->B < 0 || p->N < 1 || p->N > 64 || p->Hq < 1 || p->Hkv < 1 || p->Hq % p->Hkv != 0 || p->max_pages_per_req < 0 ||
        p->num_pages < 0 || p->kernel < 0 || p->kernel > 2 || !(p->scale > 0.f))
        return WAR_ERR_INVALID_ARG;
    // a 128-key tile is a whole number of pages, and a page is a whole number of 8-token groups of the tile layout
    if (p->D != 128 || (p->page_size != 8 && p->page_size != 16 && p->page_size != 32 && p->page_size != 64 && p->page_size != 128))
        return WAR_ERR_UNSUPPORTED;
    if ((p->Hq / p->Hkv) * p->N > 512 || p->B > kMaxPlanB) return WAR_ERR_UNSUPPORTED;
    if ((long long)p->max_pages_per_req * p->page_size >= (1ll << 30)) return WAR_ERR_UNSUPPORTED;    // contexts below 2^30 tokens
    const int layout = war_attn_pool_layout(p->k_strides, p);                 // both pools in the same one of the two layouts
    if (layout < 0 || war_attn_pool_layout(p->v_strides, p) != layout) return WAR_ERR_UNSUPPORTED;
    return WAR_OK;
}

}  // namespace

war_status_t war_attn_launch_simple(const void* q, const void* k, const void* v, const int32_t* page_table,
                                    const int32_t* prefix_len, const war_attn_params_t* p, const AttnWorkspace& w,
                                    void* out, float* lse, int* status_word, cudaStream_t s) {
    const int G = p->Hq / p->Hkv;
    const int n_sm = war_attn_sm_count();
    if (n_sm <= 0) return WAR_ERR_CUDA;
    attn_simple_kernel<<<n_sm * 4, 128, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, page_table,
                                              prefix_len, p->N, p->Hq, p->Hkv, G, p->page_size, p->max_pages_per_req,
                                              (long long)p->k_strides[0], (long long)p->k_strides[1], (long long)p->k_strides[2],
                                              (long long)p->num_pages, p->scale * kLog2e, w, (__nv_bfloat16*)out, lse, status_word);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}

extern "C" size_t war_verify_attn_workspace_bytes(const war_attn_params_t* p) {
    if (check_params(p) != WAR_OK) return 0;
    return war_attn_workspace_layout(p, nullptr).bytes;
}

extern "C" war_status_t war_verify_attn(const void* d_q, const void* d_kpool, const void* d_vpool,
                                        const int32_t* d_page_table, const int32_t* d_prefix_len,
                                        const int32_t* d_num_nodes, const int32_t* d_parent,
                                        const war_attn_params_t* p, void* d_workspace, void* d_out, float* d_lse,
                                        war_stream_t stream) {
    war_status_t st = check_params(p);
    if (st != WAR_OK) return st;
    if (p->B == 0) return WAR_OK;
    if (!d_q || !d_kpool || !d_vpool || !d_page_table || !d_prefix_len || !d_num_nodes || !d_parent || !d_workspace || !d_out)
        return WAR_ERR_INVALID_ARG;
    if (((uintptr_t)d_workspace & 255) || ((uintptr_t)d_q & 15) || ((uintptr_t)d_out & 15) || ((uintptr_t)d_kpool & 127) ||
        ((uintptr_t)d_vpool & 127))
        return WAR_ERR_INVALID_ARG;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    const AttnWorkspace w = war_attn_workspace_layout(p, d_workspace);
    const int G = p->Hq / p->Hkv;
    const int n_sm = war_attn_sm_count();
    if (n_sm <= 0) return WAR_ERR_CUDA;
    // Few requests (the low-load regime the step exists for): one launch.  Every CTA of the attention kernel plans
    // for itself and the last CTA to finish a split unit's triple merges it, so the planning and combine launches
    // and the gaps around them disappear.
    if (p->kernel == 0 && war_attn_fused_ok(p, w.row_blocks, n_sm))
        return war_attn_launch_sm100(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, d_num_nodes, d_parent, p, w, true, d_out,
                                     d_lse, status_word, stream);
    attn_plan_kernel<<<1, 1024, 0, stream>>>(d_prefix_len, d_num_nodes, d_parent, p->B, p->N, p->Hkv, G, p->page_size,
                                            p->max_pages_per_req, n_sm, w, status_word);
    WAR_LAUNCH_CHECK();
    if (p->kernel == 1)
        st = war_attn_launch_simple(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, p, w, d_out, d_lse, status_word, stream);
    else
        st = war_attn_launch_sm100(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, d_num_nodes, d_parent, p, w, false, d_out,
                                   d_lse, status_word, stream);
    if (st != WAR_OK) return st;
    attn_combine_kernel<<<dim3(p->B * p->Hkv, (G * p->N + kCombineWarps - 1) / kCombineWarps), kCombineWarps * 32, 0, stream>>>(
        w, p->N, p->Hq, p->Hkv, G, (__nv_bfloat16*)d_out, d_lse);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
