// The verify-attention plan worked out by every CTA for itself (library-internal, device code).
//
// With up to kFusedMaxB requests the work decomposition of war_attn_plan.cuh is a closed form of at most 64
// (prefix_len, num_nodes) pairs, so a separate planning launch costs more than it saves: every persistent CTA of the
// attention kernel reads those pairs, validates the trees and takes the same decisions as attn_plan_kernel
// (contiguous split, or searched chunk length + longest-first snake deal).  What stays behind is a table of a few
// hundred bytes in shared memory from which every warp role derives the CTA's next unit when it gets there; nothing
// of the plan goes through global memory.
//
// A unit of a split (request, kv head, row block) leaves its partial result in a slot of the workspace that every
// CTA can name without a table:
//   snake deal        slot = the unit's index in the longest-first list (chunk c of a triple is u0 + c * ustep)
//   contiguous split  a split pair's first chunk is the LAST unit of its CTA c0 (slot 2*c0 + 1), every further chunk
//                     is the FIRST unit of the next CTA (slot 2*(c0 + c))
// The CTA that ran chunk 0 of a split triple merges all its chunks, in chunk order, once its own units are done.
#pragma once
#include "war_attn_plan.cuh"
#include "war_common.cuh"

constexpr int kFusedMaxB = 64;
constexpr int kFusedMaxCtas = 192;          // a pair can be cut into as many chunks as there are CTAs (see kFusedMaxChunks)
constexpr int kFusedThreads = 384;
constexpr int kFusedMaxUnitsTotal = 60000;     // unit offsets are kept as 16-bit numbers

struct FusedPlan {                        // resident in shared memory for the whole kernel
    int tiles[kFusedMaxB];                // 128-key tiles per request (0: not running or rejected)
    union {
        struct {
            uint16_t pos_base[kFusedMaxB + 2];   // snake deal: first unit of the request at each sorted position
            uint16_t nc[kFusedMaxB];             // chunks per request
        } s;
        int start[kFusedMaxB + 1];        // contiguous split: first tile of each request's pairs in the sequence
    } u;
    uint8_t n[kFusedMaxB];                // validated slot count per request
    uint8_t pos_req[kFusedMaxB];          // snake deal: request at each sorted position (longest first)
    int mode;                             // 0 snake deal, 1 contiguous split
    int total;                            // snake deal: number of units
    int t_all, n_used;                    // contiguous split: tiles in the sequence, CTAs that get a range,
    int c0_first, c1_last;                //   the CTA where this CTA's first pair begins / where its last pair ends
    int lo, hi, r0, h0;                   // contiguous split: this CTA's range and the pair that holds its first tile
};
static_assert(sizeof(FusedPlan) <= 704, "the plan table shares 768 bytes of shared memory");

struct FusedPlanScratch {                 // only while the plan is made (lives in the idle ring)
    int keys[64];
    int weight[kFusedMaxB];               // units per chunk of a request: kv heads x row blocks (0: no work)
    int units_by_pos[kFusedMaxB];
    int live_before[kFusedMaxB + 1];      // contiguous split: live requests before each request
    int cut[kFusedMaxCtas + 2];           // contiguous split: first tile of every CTA's range
};

// Host-side rule for taking this path: few requests, and unit offsets that fit 16 bits (the snake deal creates at
// most kTargetUnits + one unit per (request, kv head, row block)).
inline bool war_attn_fused_ok(const war_attn_params_t* p, int row_blocks, int n_ctas) {
    return p->B <= kFusedMaxB && n_ctas <= kFusedMaxCtas && n_ctas >= 1 && p->Hkv <= 255 && p->N <= 255 &&
           (long long)p->max_pages_per_req * p->page_size < (1ll << 30) &&
           (long long)kTargetUnits + (long long)p->B * p->Hkv * row_blocks <= kFusedMaxUnitsTotal;
}

#ifdef __CUDACC__
namespace fused_plan {

struct Unit {
    int req, kvh, rb, tile_begin, tile_end, n_chunks, chunk, n_nodes;
    int slot_base, slot_stride, bump;     // partial of chunk c: slot_base + c * slot_stride (+ bump for c == 0)
};

// Walks the units of one CTA in the order they are run.  Every warp role keeps its own cursor.
struct Cursor {
    int k, r, h;
};

__device__ __forceinline__ int snake_unit(int k, int cta, int ctas) { return k * ctas + ((k & 1) ? ctas - 1 - cta : cta); }

// ceil(x / d) for 0 <= x, 0 < d, x + d <= 2^24, without an integer division
__device__ __forceinline__ int ceil_div_small(int x, int d) {
    int q = __float2int_rz(__fdividef((float)(x + d - 1), (float)d));
    const int r = (x + d - 1) - q * d;
    q += (r >= d) - (r < 0);
    return q;
}

// The chunk length for up to kFusedMaxB requests: the c in [c_lo, max(c_lo, t_max)] that minimises the estimated time
//     ceil(units(c) / CTAs) * (c + 6)  tiles,     units(c) = sum over requests of weight * ceil(tiles / c)
// (a unit costs about six tiles on top of its own: pipeline fill, Q load, partials written and merged).  Equal
// estimates take the longer chunk.  The first kThreads threads of the block evaluate one candidate each: every length
// of the range if there are that few, else every step-th one, followed by every length within a step of the best.
// Called by all threads of the block (block barriers inside); blocks of different sizes find the same length.
// `keys` is shared scratch of 64 entries.  tiles < 2^23, units(c_lo) < 2^24.
template <int kThreads>
__device__ __forceinline__ int chunk_search(const int* tiles, const int* weight, int B, int c_lo, int t_max, int n_ctas,
                                            int* keys) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int lo = c_lo, hi = max(t_max, c_lo), result = lo;
#pragma unroll 1
    while (true) {
        const int step = (hi - lo + kThreads) / kThreads;          // 1 when every length has a thread
        const int cl = min(lo + tid * step, hi);
        int est = 0x7fffffff;
        if (tid < kThreads) {
            int units = 0;                                          // (entries from B up to the next multiple of 4 have weight 0)
#pragma unroll 1
            for (int q = 0; q < B; q += 4) {
                int part[4];
#pragma unroll
                for (int k = 0; k < 4; ++k) part[k] = weight[q + k] * ceil_div_small(max(tiles[q + k], 0), cl);
                units += (part[0] + part[1]) + (part[2] + part[3]);
            }
            const int waves = ceil_div_small(units, n_ctas);
            const long long e = (long long)waves * (cl + 6);
            est = e < 0x7fffffffll ? (int)e : 0x7ffffffe;
        }
        // smallest estimate, then the longest chunk
        const int est_w = __reduce_min_sync(0xffffffffu, est);
        const int cl_w = __reduce_max_sync(0xffffffffu, est == est_w ? cl : 0);
        __syncthreads();                                            // (the previous round's keys have been read)
        if (lane == 0) { keys[2 * warp] = est_w; keys[2 * warp + 1] = cl_w; }
        __syncthreads();
        int best_e = 0x7fffffff;
        result = 0;
#pragma unroll 1
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
            const int e = keys[2 * w], c = keys[2 * w + 1];
            if (e < best_e || (e == best_e && c > result)) { best_e = e; result = c; }
        }
        if (step == 1) break;
        lo = max(lo, result - step + 1);
        hi = min(hi, result + step - 1);
    }
    return result;
}

// The contiguous split (the tiles of all (request, kv head) pairs as one sequence, cut into equal ranges, a CTA each)
// balances the CTAs to within one tile and gives every CTA at most two split units, but a range pays for an extra
// unit wherever a pair ends inside it.  Measured on 3 to 64 requests of three recipes it wins from 36-40 tiles per
// CTA on (one row block per kv head); below that the searched chunk length does better.
__host__ __device__ __forceinline__ bool contiguous_split_pays(int rows_max, long long t_all, int n_ctas) {
    return rows_max <= kRowBlock && t_all >= 36ll * n_ctas && t_all < (1ll << 30);
}

constexpr int kFusedMaxChunks = 192;      // chunks per request at most (what the merge of a row group can hold at once)
__device__ __forceinline__ int chunk_floor(int t_max) { return max(4, (t_max + kFusedMaxChunks - 1) / kFusedMaxChunks); }

// Contiguous split with the cost of a unit in it.  A CTA pays for every unit it runs about as much as for
// `unit_cost` tiles (its pipeline drains and fills again: epilogue, next Q tile, first loads; measured 12 to 21 us per
// extra unit against 1.3 us per tile, more with more query rows), so equal TILE counts leave the CTAs that hold many
// short pairs behind (finish times followed the unit count with correlation 0.9 to 0.99).  The sequence that is cut
// into equal ranges therefore gives every pair `unit_cost` virtual tiles in front of its real ones; a cut that falls
// among a pair's virtual tiles moves to the pair's first real tile.  (The constant was 8 + rows / 16 while the kernel's
// rare paths were large; with those made small a unit boundary costs about half as much: measured again on 12 to 64
// requests of three recipes, 3 to 5 + rows / 32 is 1 to 3.5 % faster than the old value.)
__host__ __device__ __forceinline__ int contiguous_unit_cost(int rows_max) { return 4 + rows_max / 32; }

// First real tile (index in the sequence of all pairs' real tiles) of CTA x's range, x in [0, n_used].
// start[r]: first real tile of request r's pairs; live_before[r]: live requests before r; weight[r] > 0: r is live.
__device__ __forceinline__ int contiguous_cut(int x, int n_used, int t_all, int pairs, int unit_cost, const int* tiles,
                                              const int* weight, const int* start, const int* live_before, int B, int Hkv) {
    if (x >= n_used) return t_all;
    // position in the weighted sequence, floor(w_all * x / n_used), in 32-bit arithmetic (w_all < 2^31, x < 2^10)
    const unsigned w_all = (unsigned)t_all + (unsigned)(pairs * unit_cost);
    const unsigned base = w_all / (unsigned)n_used, rem = w_all - base * (unsigned)n_used;
    const unsigned p = base * (unsigned)x + rem * (unsigned)x / (unsigned)n_used;
    // The request whose pairs hold weighted position p: the last live one that starts at or before it.  Weighted starts
    // do not decrease with the request index (a request that is not live starts where the next live one does), the
    // first is 0 and p lies below the end of the sequence, so the last index that starts at or before p is a live
    // request: a binary search (this runs in every CTA of the one-launch path, for every cut, before the first copy).
    int r = 0, top = B - 1;
#pragma unroll 1
    while (r < top) {
        const int mid = (r + top + 1) >> 1;
        if ((unsigned)(start[mid] + live_before[mid] * Hkv * unit_cost) <= p) r = mid; else top = mid - 1;
    }
    if (weight[r] <= 0) {                                            // (not reached: see above)
        r = -1;
#pragma unroll 1
        for (int q = 0; q < B; ++q)
            if (weight[q] > 0 && (unsigned)(start[q] + live_before[q] * Hkv * unit_cost) <= p) r = q;
        if (r < 0) return 0;
    }
    const unsigned off = p - (unsigned)(start[r] + live_before[r] * Hkv * unit_cost);
    const unsigned w = (unsigned)(tiles[r] + unit_cost);
    const int h = (int)(off / w);
    if (h >= Hkv) return start[r] + Hkv * tiles[r];              // (cannot happen: the next live request starts there)
    const int o = (int)(off - (unsigned)h * w);
    return start[r] + h * tiles[r] + max(0, o - unit_cost);
}

__device__ __forceinline__ void cursor_init(const FusedPlan* pl, Cursor& c) { c.k = 0; c.r = pl->r0; c.h = pl->h0; }

// The CTA's next unit (false: none left).
__device__ __forceinline__ bool next_unit(const FusedPlan* pl, Cursor& c, int B, int Hkv, int G, Unit& un) {
    const int cta = blockIdx.x, n_ctas = gridDim.x;
    if (pl->mode == 0) {
        const int u = snake_unit(c.k, cta, n_ctas);
        if (u >= pl->total) return false;
        int lo = 0, hi = B - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if ((int)pl->u.s.pos_base[mid] <= u) lo = mid; else hi = mid - 1;
        }
        const int i = pl->pos_req[lo];
        const int t = pl->tiles[i], n = pl->n[i], nc = pl->u.s.nc[i];
        const int rbs = (G * n + kRowBlock - 1) / kRowBlock;
        const int local = u - (int)pl->u.s.pos_base[lo];
        const int per = Hkv * rbs;
        const int ch = local / per, rem = local - ch * per;
        un.req = i; un.kvh = rem / rbs; un.rb = rem - un.kvh * rbs; un.n_nodes = n;
        if (t < 32768 && nc < 32768) {
            un.tile_begin = (int)((unsigned)t * (unsigned)ch / (unsigned)nc); un.tile_end = (int)((unsigned)t * (unsigned)(ch + 1) / (unsigned)nc);
        } else {
            un.tile_begin = (int)((long long)t * ch / nc); un.tile_end = (int)((long long)t * (ch + 1) / nc);
        }
        un.n_chunks = nc; un.chunk = ch;
        un.slot_base = u - ch * per; un.slot_stride = per; un.bump = 0;
        ++c.k;
        return true;
    }
    // contiguous split: the pairs that overlap [lo, hi), one after the other
    const int lo = pl->lo, hi = pl->hi;
    if (c.r >= B) return false;
    const int t = pl->tiles[c.r];
    const int ps = pl->u.start[c.r] + c.h * t;
    if (ps >= hi) return false;
    // only a CTA's first unit can have begun in an earlier CTA, only its last one can go on into a later one
    const int c0 = ps >= lo ? cta : pl->c0_first, c1 = ps + t <= hi ? cta : pl->c1_last;
    un.req = c.r; un.kvh = c.h; un.rb = 0; un.n_nodes = pl->n[c.r];
    un.tile_begin = max(lo, ps) - ps; un.tile_end = min(hi, ps + t) - ps;
    un.n_chunks = c1 - c0 + 1; un.chunk = cta - c0;
    un.slot_base = 2 * c0; un.slot_stride = 2; un.bump = 1;
    ++c.k;
    if (++c.h == Hkv) {
        c.h = 0;
        do { ++c.r; } while (c.r < B && (pl->n[c.r] == 0 || pl->tiles[c.r] <= 0));
    }
    return true;
}

// Executed by all kFusedThreads threads of the CTA (it contains block barriers).  The code below runs once per CTA
// and launch, straight from a cold instruction cache, so its cost is its length: it reads only the two numbers per
// request the plan depends on (the parent arrays are checked by the warps that use them, unit by unit), keeps to
// 32-bit arithmetic and rolled loops, and has two block barriers on the contiguous path and five on the other.
__device__ __noinline__ static void make(const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ num_nodes,
                                        int B, int N, int Hkv, int G, int page_size, int max_pages,
                                        FusedPlanScratch* sc, FusedPlan* pl, int* status_word) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_ctas = gridDim.x, cta = blockIdx.x;
    if (tid < kFusedMaxB) {
        int n = 0, tiles = 0;
        if (tid < B) {
            n = num_nodes[tid];
            const int pfx = prefix_len[tid];
            if (n < 0 || n > N || pfx < 0) { war_set_device_status(status_word, WAR_ERR_BAD_TREE); n = 0; }
            if (n > 0) {
                const long long L = (long long)pfx + n;
                if (L > (long long)max_pages * page_size) { war_set_device_status(status_word, WAR_ERR_BAD_PAGE); n = 0; }
                else tiles = (int)((L + kTileKeys - 1) >> 7);
            }
        }
        pl->tiles[tid] = tiles;
        pl->n[tid] = (uint8_t)n;
        sc->weight[tid] = n > 0 && tiles > 0 ? Hkv * ((G * n + kRowBlock - 1) / kRowBlock) : 0;
    }
    __syncthreads();

    // ---- the same choice as attn_plan_kernel makes for up to 64 requests (every warp for itself) ----
    int n_mx = 0, prs = 0, t_mx = 0, t_sm = 0;
    long long w_sm = 0;
    for (int q = lane; q < B; q += 32) {
        const int w = sc->weight[q], t = pl->tiles[q];
        if (w > 0) { n_mx = max(n_mx, (int)pl->n[q]); prs += Hkv; t_mx = max(t_mx, t); t_sm += t; w_sm += (long long)t * w; }
    }
    const int rows_max = G * __reduce_max_sync(0xffffffffu, n_mx);
    const int pairs = __reduce_add_sync(0xffffffffu, prs);
    const int t_max = __reduce_max_sync(0xffffffffu, t_mx);
    const int t_sum = __reduce_add_sync(0xffffffffu, t_sm);
    // all tiles, weighted by kv heads and row blocks (the sum of the lanes' numbers in two 32-bit pieces)
    const long long tot = ((long long)__reduce_add_sync(0xffffffffu, (unsigned)(w_sm >> 24)) << 24) +
                          (long long)__reduce_add_sync(0xffffffffu, (unsigned)(w_sm & 0xffffff));
    const long long t_all_ll = (long long)t_sum * Hkv;
    const bool contiguous = contiguous_split_pays(rows_max, t_all_ll, n_ctas);

    if (contiguous) {
        // The tiles of all (request, kv head) pairs form one sequence; CTA c takes [cut(c), cut(c+1)) (contiguous_cut).
        if (warp == 0) {
            const int a0 = 2 * lane, a1 = 2 * lane + 1;
            const int l0 = sc->weight[a0] > 0, l1 = sc->weight[a1] > 0;
            const int m0 = l0 ? pl->tiles[a0] * Hkv : 0, m1 = l1 ? pl->tiles[a1] * Hkv : 0;
            int incl = m0 + m1, live = l0 + l1;
#pragma unroll 1
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, incl, o), z = __shfl_up_sync(0xffffffffu, live, o);
                if (lane >= o) { incl += y; live += z; }
            }
            pl->u.start[a0] = incl - m0 - m1;
            pl->u.start[a1] = incl - m1;
            sc->live_before[a0] = live - l0 - l1;
            sc->live_before[a1] = live - l1;
            if (lane == 31) {
                pl->u.start[64] = incl;
                pl->mode = 1; pl->total = 0; pl->t_all = incl; pl->n_used = min(n_ctas, max(1, incl / 4));
            }
        }
        __syncthreads();
        const int t_all = pl->t_all, n_used = pl->n_used;
        const int unit_cost = contiguous_unit_cost(rows_max);
        for (int x = tid; x <= n_used; x += kFusedThreads)
            sc->cut[x] = contiguous_cut(x, n_used, t_all, pairs, unit_cost, pl->tiles, sc->weight, pl->u.start, sc->live_before, B, Hkv);
        __syncthreads();
        if (warp == 0) {
            // this CTA's range, the pair that holds its first tile (lanes look at requests lane and lane + 32), and the
            // CTAs where its first pair begins and its last pair ends (lanes look at cuts lane, lane + 32, ...)
            int lo = 0, hi = 0;
            if (cta < n_used) { lo = sc->cut[cta]; hi = sc->cut[cta + 1]; }
            int best = -1;
            for (int q = lane; q < B; q += 32)
                if (sc->weight[q] > 0 && pl->u.start[q] <= lo) best = max(best, q);
            best = __reduce_max_sync(0xffffffffu, best);
            int r0 = B, h0 = 0, c0_first = cta, c1_last = cta;
            if (hi > lo && best >= 0) {
                r0 = best; h0 = (int)((unsigned)(lo - pl->u.start[best]) / (unsigned)pl->tiles[best]);
                const int ps0 = pl->u.start[r0] + h0 * pl->tiles[r0];        // first tile of the pair that holds lo
                int last = -1;                                               // the pair that holds hi - 1, and its last tile
                for (int q = lane; q < B; q += 32)
                    if (sc->weight[q] > 0 && pl->u.start[q] <= hi - 1) last = max(last, q);
                last = __reduce_max_sync(0xffffffffu, last);
                const int hl = (int)((unsigned)(hi - 1 - pl->u.start[last]) / (unsigned)pl->tiles[last]);
                const int pe = pl->u.start[last] + (hl + 1) * pl->tiles[last] - 1;
                // the CTA whose non-empty range holds a tile: the largest x with cut[x] <= tile and cut[x + 1] > tile
                int f = -1, l = -1;
                for (int x = lane; x < n_used; x += 32) {
                    if (sc->cut[x] <= ps0 && sc->cut[x + 1] > ps0) f = x;
                    if (sc->cut[x] <= pe && sc->cut[x + 1] > pe) l = x;
                }
                c0_first = __reduce_max_sync(0xffffffffu, f);
                c1_last = __reduce_max_sync(0xffffffffu, l);
            }
            if (lane == 0) { pl->lo = lo; pl->hi = hi; pl->r0 = r0; pl->h0 = h0; pl->c0_first = c0_first; pl->c1_last = c1_last; }
        }
        __syncthreads();
        return;
    }

    // ---- searched chunk length (see chunk_search), never more than kFusedMaxChunks chunks per request ----
    long long ct = (tot + kTargetUnits - 1) / kTargetUnits;
    if (ct < kMinChunkTiles) ct = kMinChunkTiles;
    const int chunk_tiles = (int)ct;
    const int best_c = chunk_search<kFusedThreads>(pl->tiles, sc->weight, B, max(chunk_floor(t_max), chunk_tiles), t_max, n_ctas, sc->keys);
    const int c_best = best_c;
    // ---- longest-first order, units per request, their offsets ----
    if (tid < B) {
        const int t = pl->tiles[tid];
        int pos = 0;
        for (int q = 0; q < B; ++q) {
            const int tq = pl->tiles[q];
            pos += (tq > t) || (tq == t && q < tid);
        }
        const int nc = t > 0 ? ceil_div_small(t, c_best) : 0;
        pl->u.s.nc[tid] = (uint16_t)nc;
        pl->pos_req[pos] = (uint8_t)tid;
        sc->units_by_pos[pos] = nc * sc->weight[tid];
        sc->live_before[pos] = nc > 1 ? sc->weight[tid] : 0;      // (idle in this mode) split triples of the request
    }
    __syncthreads();
    if (warp == 0) {                                             // exclusive scan over the sorted positions, two per lane
        const int a0 = 2 * lane, a1 = 2 * lane + 1;
        const int m0 = a0 < B ? sc->units_by_pos[a0] : 0, m1 = a1 < B ? sc->units_by_pos[a1] : 0;
        int incl = m0 + m1;
#pragma unroll 1
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
        pl->u.s.pos_base[a0] = (uint16_t)(incl - m0 - m1);
        pl->u.s.pos_base[a1] = (uint16_t)(incl - m1);
        const int split = __reduce_add_sync(0xffffffffu, (a0 < B ? sc->live_before[a0] : 0) + (a1 < B ? sc->live_before[a1] : 0));
        // (in this mode n_used holds the number of split (request, kv head, row block) triples and t_all the largest
        // number of rows of a row block, for the deal of the merges)
        if (lane == 31) { pl->mode = 0; pl->total = incl; pl->r0 = 0; pl->h0 = 0; pl->lo = 0; pl->hi = 0; pl->t_all = min(rows_max, kRowBlock); pl->n_used = split; pl->c0_first = 0; pl->c1_last = 0; }
    }
    __syncthreads();
}

}  // namespace fused_plan
#endif
