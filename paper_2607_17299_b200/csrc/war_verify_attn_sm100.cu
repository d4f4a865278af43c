// Tensor-core verify attention for sm_100a: TMA-staged KV pages -> tcgen05.mma with accumulators in TMEM ->
// online softmax -> tcgen05.mma again, one persistent CTA per SM.
//
// Work unit (see war_attn_plan.cuh): up to 128 query rows (slot, head-of-group) of one kv head against a range of
// 128-key tiles.  Per tile:   S = Q K^T   (M=128 rows, N=128 keys, K=128 dims; bf16 operands in shared memory)
//                             P = exp2(S*scale*log2e - m), masked by the tree's ancestor bits on tree columns
//                             O += P V    (M=128 rows, N=128 dims, K=128 keys; P is read from TMEM)
// Tiles alternate between two softmax groups, each with its own S/P region, running (max, sum) and O accumulator
// in TMEM; the two partial results are merged once per unit.  Nothing synchronises the groups per tile.
// Warp roles:  warp 8   producer: reads the page table, issues one TMA tensor copy per (page, head) into a ring of
//                       32 KB slots in the order the tensor pipe consumes them (K0 K1 V0 K2 V1 ...); every CTA loads for itself,
//                       this GPU's memory only
//              warp 9   MMA issuer (one lane): S(t+2) is queued right behind PV(t); owns the TMEM allocation
//              warps 0-3 / 4-7  softmax group 0 / 1: one thread per query row (TMEM lane); the whole row of S is
//                       pulled into registers once, P goes back into the first 64 columns of the same TMEM region
//                       as packed bf16; O is rescaled in TMEM only when the running max grows by more than 2^8
//              The softmax warpgroups take registers from the third one (setmaxnreg) so a row of S fits.
// Shared-memory operand layouts are the canonical 128-byte-swizzled ones: K-major for Q and K, MN-major for V.
// Head-major pools: a (page, head) block lands as [token/8][d/64][token%8][d%64], which serves both K (K-major,
// 8-row groups 2 KB apart) and V (MN-major, 64-wide column blocks 1 KB apart, 8-key groups 2 KB apart) with one
// copy per block.  Token-major pools (a page stored as [token][head][d]) cannot be copied that way in one piece (it
// would take a 6-dimensional tensor map), so there a tile is laid out as [d/64][token][d%64] (8-row groups 1 KB
// apart, the two 64-wide halves 16 KB apart) and every (page, head) takes two copies, one per half.
// Every wait is bounded: on expiry the kernel records WAR_ERR_TIMEOUT, raises a CTA-wide abort flag and returns.
// With up to 64 requests the same kernel also plans and merges (template parameter kFused): one launch per call.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>
#include <atomic>
#include <chrono>
#include <mutex>
#include "war_common.cuh"
#include "war_attn_plan.cuh"
#include "war_attn_fused_plan.cuh"
#include "war_sm100_prims.cuh"

namespace {
using namespace sm100;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kSlots = 6;
constexpr int kSlotBytes = 32768;
constexpr int kThreads = 384;                      // three warpgroups: softmax 0, softmax 1, {producer, MMA, 2 spare warps}
constexpr int kRegsSoftmax = 224;                   // register budget after the hand-over below
constexpr int kRegsOther = 48;
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;           // log2 units

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffRing = 32768;
constexpr int kOffBar = kOffRing + kSlots * kSlotBytes;
constexpr int kOffStats = kOffBar + 256;
constexpr int kOffFused = kOffStats + 1024;          // fused-plan variant only: this CTA's unit list
constexpr int kSmemBytes = kOffStats + 1024 + 1024;
constexpr int kSmemBytesFused = kOffFused + 768 + 1024;
static_assert(sizeof(FusedPlan) <= 768, "plan table of the fused-plan variant");
static_assert(kSmemBytesFused <= 232448, "shared memory of the fused-plan variant");
static_assert(sizeof(FusedPlanScratch) <= kSlots * kSlotBytes, "the plan scratch lives in the idle ring");
static_assert(kThreads == kFusedThreads, "fused_plan::make is written for the attention kernel's block size");

struct Bars {
    uint64_t full[kSlots], empty[kSlots];
    uint64_t s_ready[2], p_ready[2], pv_done[2];
    uint64_t q_ready, stats_ready, epi_done;
    uint64_t part_out;                   // fused-plan variant: a split unit's partial has been written (128 arrivals)
    uint64_t merge_full, merge_free;     // fused-plan variant: a row group's partials have landed / have been read
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(Bars) <= 256, "barrier block");

// Ring sequence numbers inside a unit of T tiles whose first load has number ld0.  Loads are issued in the order
// the tensor pipe consumes them: K0, K1, V0, K2, V1, ..., K(T-1), V(T-2), V(T-1).
__device__ __forceinline__ uint32_t seq_k(uint32_t ld0, int t) { return t == 0 ? ld0 : ld0 + 2u * t - 1u; }
__device__ __forceinline__ uint32_t seq_v(uint32_t ld0, int t, int T) { return t == T - 1 ? ld0 + 2u * T - 1u : ld0 + 2u * t + 2u; }

struct KernelArgs {
    const __nv_bfloat16* q;
    const int32_t* page_table;
    const int32_t* prefix_len;
    __nv_bfloat16* out;
    float* lse;
    int* status_word;
    AttnWorkspace w;
    long long num_pages;
    float scale_log2;
    int N, Hq, Hkv, G, page_size, max_pages;
    // fused-plan variant
    const int32_t* num_nodes;
    const int32_t* parent;
    int B;
    unsigned long long call;             // number of this launch (48 bits, never 0)
};

// What the three roles need to know about a unit, wherever the plan lives.
struct UnitView {
    int req, kvh, rb, tile_begin, tile_end, n_chunks, chunk, n_nodes;
    int slot;                            // index of this unit's partial in the workspace
    int slot_base, slot_stride, bump;    // fused-plan variant: partial of chunk c is slot_base + c * slot_stride (+ bump for c == 0)
};

// Ancestor-or-self bit masks of one tree, by one warp: lane l holds slots l and l + 32.  After round r a slot's mask
// covers its 2^r nearest ancestors-or-self and its pointer is the 2^r-th ancestor (the root points at itself).
// Returns the mask of slot j (any j < n per lane).  The tree has been validated (parent[s] in [0, s) for 0 < s < n).
__device__ __forceinline__ uint64_t shfl_u64(uint64_t v, int src) {
    const uint32_t lo = __shfl_sync(0xffffffffu, (uint32_t)v, src);
    const uint32_t hi = __shfl_sync(0xffffffffu, (uint32_t)(v >> 32), src);
    return ((uint64_t)hi << 32) | lo;
}
// parent[s] must lie in [0, s) for every slot 0 < s < n (lane l holds the entries of slots l and l + 32)
__device__ __forceinline__ bool tree_is_malformed(int q0, int q1, int n, int lane) {
    const int j0 = lane, j1 = lane + 32;
    const bool bad = (j0 > 0 && j0 < n && (q0 < 0 || q0 >= j0)) || (j1 < n && (q1 < 0 || q1 >= j1));
    return __any_sync(0xffffffffu, bad);
}
__device__ __forceinline__ uint64_t warp_ancestor_mask(int q0, int q1, int n, int j, int lane) {
    const int j0 = lane, j1 = lane + 32;
    int p0 = (j0 > 0 && j0 < n) ? q0 : 0;
    int p1 = (j1 < n) ? q1 : 0;
    uint64_t a0 = 1ull << j0, a1 = 1ull << j1;
    // (rolled loops: this runs once per unit, from code that is usually not in the instruction cache)
    if (n <= 32) {
#pragma unroll 1
        for (int r = 0; r < 5; ++r) {
            const uint64_t b = shfl_u64(a0, p0);
            const int q = __shfl_sync(0xffffffffu, p0, p0);
            a0 |= b; p0 = q;
        }
    } else {
#pragma unroll 1
        for (int r = 0; r < 6; ++r) {
            const uint64_t b00 = shfl_u64(a0, p0 & 31), b01 = shfl_u64(a1, p0 & 31);
            const uint64_t b10 = shfl_u64(a0, p1 & 31), b11 = shfl_u64(a1, p1 & 31);
            const int q00 = __shfl_sync(0xffffffffu, p0, p0 & 31), q01 = __shfl_sync(0xffffffffu, p1, p0 & 31);
            const int q10 = __shfl_sync(0xffffffffu, p0, p1 & 31), q11 = __shfl_sync(0xffffffffu, p1, p1 & 31);
            a0 |= p0 >= 32 ? b01 : b00;
            a1 |= p1 >= 32 ? b11 : b10;
            p0 = p0 >= 32 ? q01 : q00;
            p1 = p1 >= 32 ? q11 : q10;
        }
    }
    const uint64_t m0 = shfl_u64(a0, j & 31), m1 = shfl_u64(a1, j & 31);
    return j >= 32 ? m1 : m0;
}

// Arrival counters of split (request, kv head, row block) triples (fused-plan variant).  A word holds
// (call number << 16) | arrivals (one per unit, at most kFusedMaxChunks).  The call number (48 bits, never 0, a new
// one for every launch made by this process) makes a word written by an earlier call, or never written at all, read
// as "no arrivals yet", so nothing has to be cleared before a launch; the CTA that merges a triple writes 0 back, so
// a captured launch (whose call number is frozen in the graph) can be replayed.  (A word that was never written
// equals the current call number by accident with probability 2^-48.)
__device__ __forceinline__ void count_arrival(unsigned long long* p, unsigned long long call) {
    const unsigned long long old = atomicAdd(p, 1ull);
    if ((old >> 16) == call) return;                         // the usual case after a triple's first arrival
    // The word was not this call's: the increment above went to a stale word and does not count.  Either make the
    // word this call's with one arrival, or, if somebody else has done so meanwhile, add this arrival to it.
    unsigned long long cur = old + 1ull;
    while (true) {
        if ((cur >> 16) == call) { atomicAdd(p, 1ull); return; }
        const unsigned long long prev = atomicCAS(p, cur, (call << 16) | 1ull);
        if (prev == cur) return;
        cur = prev;
    }
}
// The same count that also says how many of this call's arrivals there are now, this one included.
__device__ __noinline__ int count_arrival_ranked(unsigned long long* p, unsigned long long call) {
    const unsigned long long old = atomicAdd(p, 1ull);
    if ((old >> 16) == call) return (int)(old & 0xffffull) + 1;
    unsigned long long cur = old + 1ull;
    while (true) {
        if ((cur >> 16) == call) return (int)(atomicAdd(p, 1ull) & 0xffffull) + 1;
        const unsigned long long prev = atomicCAS(p, cur, (call << 16) | 1ull);
        if (prev == cur) return 1;
        cur = prev;
    }
}
// Bounded wait (one thread) until `target` arrivals of this call have been counted in p[0]; then the word is cleared.
// When `parts` CTAs merge the triple, each a share of its rows, every one of them waits here; they count themselves
// in *seen once they have seen the arrivals, and the last one to do so clears both words.
template <class BarsT>
__device__ __forceinline__ bool wait_arrivals(unsigned long long* p, unsigned long long* seen, unsigned long long call, int target, int parts, BarsT* bars, int* status_word) {
    auto there = [&]() -> bool {
        unsigned long long v;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
        return (v >> 16) == call && (int)(v & 0xffffull) >= target;
    };
    if (!there()) {
        const unsigned long long t0 = global_timer_ns();
        unsigned spins = 0;
        while (!there()) {
            if ((++spins & 63u) == 0) {
                if (*(volatile int*)&bars->abort_flag) return false;
                if (global_timer_ns() - t0 > kWaitBudgetNs) {
                    war_set_device_status(status_word, WAR_ERR_TIMEOUT);
                    atomicExch(&bars->abort_flag, 1);
                    return false;
                }
            }
        }
    }
    __threadfence();
    if (parts > 1) {
        if (count_arrival_ranked(seen, call) < parts) return true;
        *(volatile unsigned long long*)seen = 0ull;
    }
    *(volatile unsigned long long*)p = 0ull;
    return true;
}

// Merge of the partial results of one split (request, kv head, row block) by the CTA that ran its chunk 0
// (fused-plan variant), once all units of the CTA are done and the ring and the Q tile are idle.  The eight softmax
// warps call it together.  Rows are taken in groups small enough that every chunk's rows of a group fit the ring at
// once: one thread issues a bulk copy per chunk for the partial outputs (ring) and one for the (max, sum) pairs (Q
// tile), everybody waits for the bytes, then every warp takes rows of the group, four at a time: row maximum over
// the chunks, then the chunks in chunk order with the arithmetic of attn_combine_kernel, so the bits do not depend
// on who merges.  Loops are rolled on purpose: this code runs once or twice per launch from a cold instruction cache.
// `phase` counts the groups this CTA has merged so far (the parity of both barriers).
struct MergeArgs {
    const float* part_o; const float* part_ml;
    __nv_bfloat16* out; float* lse; int* status_word;
    int rows, G, N, Hq;
    int req, kvh, rb, n_nodes, n_chunks, slot_base, slot_stride, bump;
    int part, parts, share;              // this CTA merges share `part` of `parts`: rows [part * share, + share), share even
    unsigned long long* arrivals; unsigned long long* seen; unsigned long long call;
};
template <class BarsT>
__device__ __noinline__ bool merge_partials(const MergeArgs m, uint8_t* smem, BarsT* bars, uint32_t* phase_io) {
    const int tid = threadIdx.x, w8 = tid >> 5, lane = tid & 31;
    const int R = m.G * m.n_nodes;
    const int rows_valid = min(kRowBlock, R - m.rb * kRowBlock);
    const int nch = m.n_chunks;
    uint32_t phase = *phase_io;
    const int rows_g = min(kRowBlock, ((kSlots * kSlotBytes) / (nch * 512)) & ~1);     // even, >= 2 (nch <= kFusedMaxChunks)
    const float* s_o = (const float*)(smem + kOffRing);
    const float2* s_ml = (const float2*)(smem + kOffQ);
    int r_lo = 0, r_hi = rows_valid;
    if (m.parts > 1) {
        r_lo = m.part * m.share; r_hi = min(rows_valid, r_lo + m.share);
        if (r_lo >= r_hi) {                   // nothing falls to this share; it still takes part in clearing the counter
            if (tid == 0 && !wait_arrivals(m.arrivals, m.seen, m.call, nch, m.parts, bars, m.status_word)) return false;
            return true;
        }
    }
    for (int row0 = r_lo; row0 < r_hi; row0 += rows_g, ++phase) {
        const int rg = min(rows_g, (r_hi - row0 + 1) & ~1);                           // rows copied (even; the workspace has them)
        if (tid == 0) {
            // every chunk has left its partial
            if (row0 == r_lo && !wait_arrivals(m.arrivals, m.seen, m.call, nch, m.parts, bars, m.status_word)) { *phase_io = phase; return false; }
            // the previous group's readers are done with the buffers
            if (phase > 0 && !mbar_wait(&bars->merge_free, (phase - 1) & 1u, bars, m.status_word)) { *phase_io = phase; return false; }
            mbar_arrive_expect_tx(&bars->merge_full, (uint32_t)(nch * rg * (512 + 8)));
            for (int c = 0; c < nch; ++c) {
                const size_t slot = (size_t)(m.slot_base + c * m.slot_stride + (c == 0 ? m.bump : 0));
                const size_t at = slot * m.rows + row0;
                bulk_load(smem_u32(s_o + (size_t)c * rg * 128), m.part_o + at * 128, (uint32_t)rg * 512u, &bars->merge_full);
                bulk_load(smem_u32(s_ml + (size_t)c * rg), m.part_ml + at * 2, (uint32_t)rg * 8u, &bars->merge_full);
            }
        }
        if (!mbar_wait(&bars->merge_full, phase & 1u, bars, m.status_word)) { *phase_io = phase; return false; }
        // a warp takes four rows at a time, eight lanes per row, each lane four float4 of the row (columns 4*sub + 32*k):
        // sixteen independent accumulators per lane, and a load instruction reads four whole 128-byte segments
        const int sub = lane & 7;
        for (int rbase = w8 * 4; rbase < rg; rbase += 32) {
            const int r = rbase + (lane >> 3);
            const bool live = r < rg && row0 + r < r_hi;
            const int rr = live ? r : 0;
            float M = -CUDART_INF_F;
#pragma unroll 1
            for (int c = 0; c < nch; ++c) M = fmaxf(M, s_ml[c * rg + rr].x);
            float l = 0.f;
            float4 acc[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
            for (int c = 0; c < nch; ++c) {
                const float2 ml = s_ml[c * rg + rr];
                const float4* src = reinterpret_cast<const float4*>(s_o + ((size_t)c * rg + rr) * 128) + sub;
                const float sc = ml.x == -CUDART_INF_F ? 0.f : exp2f(ml.x - M);
                l = fmaf(ml.y, sc, l);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float4 o = src[8 * k];
                    acc[k].x = fmaf(o.x, sc, acc[k].x); acc[k].y = fmaf(o.y, sc, acc[k].y);
                    acc[k].z = fmaf(o.z, sc, acc[k].z); acc[k].w = fmaf(o.w, sc, acc[k].w);
                }
            }
            if (live) {
                const int gr = m.rb * kRowBlock + row0 + r;
                const int j = gr / m.G, g = gr - j * m.G;
                const size_t row = ((size_t)m.req * m.N + j) * m.Hq + m.kvh * m.G + g;
                const float inv = 1.f / l;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[k].x * inv, acc[k].y * inv), h1 = __floats2bfloat162_rn(acc[k].z * inv, acc[k].w * inv);
                    uint2 packed;
                    packed.x = *reinterpret_cast<const uint32_t*>(&h0);
                    packed.y = *reinterpret_cast<const uint32_t*>(&h1);
                    *reinterpret_cast<uint2*>(m.out + row * 128 + (sub + 8 * k) * 4) = packed;
                }
                if (m.lse && sub == 0) m.lse[row] = (M + log2f(l)) * kLn2;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->merge_free);
    }
    *phase_io = phase;
    return true;
}

// kTokenMajor: pool layout, false = (page, head, token, d), true = (page, token, head, d).
// kFused: false = the plan comes from attn_plan_kernel through the workspace and attn_combine_kernel merges split
// units afterwards; true = every CTA works its own units out (war_attn_fused_plan.cuh), a spare warp counts the split
// units whose partials are out, and once a CTA is through its units its softmax warps merge the split triples that
// fall to it (waiting, with a bound, for their last chunk), so the call is one launch.
template <bool kTokenMajor, bool kFused>
__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const KernelArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Bars* bars = (Bars*)(smem + kOffBar);
    float2* stats = (float2*)(smem + kOffStats);     // group 1's (max, sum) per row, for the merge
    const FusedPlan* plan = (const FusedPlan*)(smem + kOffFused);
    const uint32_t sQ = smem_u32(smem + kOffQ), sRing = smem_u32(smem + kOffRing);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int n_units = 0, list_first = 0, list_end = 0;
    bool contiguous = false;
    if (!kFused) {
        n_units = a.w.counters[1];
        // k-th unit of this CTA: its own contiguous list, or the snake deal of the longest-first list
        contiguous = a.w.counters[3] != 0 && gridDim.x <= (unsigned)kMaxPlanCtas;
        list_first = contiguous ? a.w.cta_first[blockIdx.x] : 0; list_end = contiguous ? a.w.cta_first[blockIdx.x + 1] : 0;
    }
    auto unit_at = [&](int k) -> int {
        if (contiguous) return list_first + k < list_end ? list_first + k : n_units;
        return snake_unit(k, blockIdx.x, gridDim.x);
    };
    // next unit of this CTA (false: no more); every warp role walks the list with its own cursor
    auto fetch = [&](fused_plan::Cursor& cur, UnitView& un) -> bool {
        if (kFused) {
            fused_plan::Unit f;
            if (!fused_plan::next_unit(plan, cur, a.B, a.Hkv, a.G, f)) return false;
            un.req = f.req; un.kvh = f.kvh; un.rb = f.rb; un.n_nodes = f.n_nodes;
            un.tile_begin = f.tile_begin; un.tile_end = f.tile_end; un.n_chunks = f.n_chunks; un.chunk = f.chunk;
            un.slot_base = f.slot_base; un.slot_stride = f.slot_stride; un.bump = f.bump;
            un.slot = f.slot_base + f.chunk * f.slot_stride + (f.chunk == 0 ? f.bump : 0);
            return true;
        }
        const int u = unit_at(cur.k++);
        if (u >= n_units) return false;
        const AttnUnit x = a.w.units[u];
        un.req = x.req; un.kvh = x.kvh; un.rb = x.rb; un.tile_begin = x.tile_begin; un.tile_end = x.tile_end;
        un.n_chunks = x.n_chunks; un.chunk = x.chunk; un.n_nodes = a.w.req[x.req].n_nodes;
        un.slot = u; un.slot_base = 0; un.slot_stride = 0; un.bump = 0;
        return true;
    };
    const int pages_per_tile = kTileKeys / a.page_size;
    const uint32_t page_bytes = (uint32_t)a.page_size * 256u;

    if (tid == 0) {
        for (int i = 0; i < kSlots; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&bars->s_ready[i], 1); mbar_init(&bars->p_ready[i], 128); mbar_init(&bars->pv_done[i], 1); }
        mbar_init(&bars->q_ready, 256);
        mbar_init(&bars->stats_ready, 128);
        mbar_init(&bars->epi_done, 128);
        mbar_init(&bars->part_out, 128);
        mbar_init(&bars->merge_full, 1);
        mbar_init(&bars->merge_free, 8);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (kFused) {
        // this CTA's units, worked out here (the ring is idle until the first unit starts)
        fused_plan::make(a.prefix_len, a.num_nodes, a.B, a.N, a.Hkv, a.G, a.page_size, a.max_pages,
                         (FusedPlanScratch*)(smem + kOffRing), (FusedPlan*)(smem + kOffFused), a.status_word);
    }
    if (kFused) fence_async_proxy();                       // the plan's scratch is about to be overwritten by tensor copies
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = bars->tmem_base;
    // columns: [0,128) S/P of group 0, [128,256) S/P of group 1, [256,384) O of group 0, [384,512) O of group 1

    // register hand-over between warpgroups: the third warpgroup gives registers up, the softmax warpgroups take them
    // (each instruction is executed by all four warps of its warpgroup, and the role code stays inside that branch)
    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (warp == 8) {
        // ------------------------------------------------------------------ producer
        // One-launch variant (64 requests or fewer), one row block per kv head: every K/V line is read once per call,
        // by one CTA, and is marked to leave L2 first, so that the stream does not push out what the step reads again
        // (the index the draft kernel probes, page tables, the kernels' own code).  With several row blocks the
        // siblings share K/V through L2 and the lines keep the default policy; so do the large batches of the
        // three-launch variant, where the mark bought nothing and cost 2-3 %.
        const bool stream_once = kFused && a.w.row_blocks == 1;
        const uint64_t evict_first = kFused ? l2_policy_evict_first() : 0ull;
        uint32_t ld = 0;
        bool ok = true;
        fused_plan::Cursor cur{0, 0, 0};
        if (kFused) fused_plan::cursor_init(plan, cur);
        while (ok) {
            UnitView un;
            if (!fetch(cur, un)) break;
            const int i = un.req;
            const int L = a.prefix_len[i] + un.n_nodes;
            const int total_pages = (L + a.page_size - 1) / a.page_size;
            const int32_t* pt = a.page_table + (size_t)i * a.max_pages;
            const int T = un.tile_end - un.tile_begin;
            auto page_of = [&](int t) -> int {                   // this lane's page id in local tile t (-1: none)
                if (t >= T || lane >= pages_per_tile) return -1;
                const int pi = (un.tile_begin + t) * pages_per_tile + lane;
                return pi < total_pages ? pt[pi] : -1;
            };
            auto load = [&](int t, int page, bool is_v) -> bool {
                const uint32_t slot = ld % kSlots, phase = (ld / kSlots) & 1u;
                ++ld;
                bool w = mbar_wait(&bars->empty[slot], phase ^ 1u, bars, a.status_word);
                w = __all_sync(0xffffffffu, w);
                if (!w) return false;
                const int n_valid = min(pages_per_tile, total_pages - (un.tile_begin + t) * pages_per_tile);
                if (lane == 0) mbar_arrive_expect_tx(&bars->full[slot], (uint32_t)n_valid * page_bytes);
                __syncwarp();
                if (lane < n_valid) {
                    long long pg = page;
                    if (pg < 0 || pg >= a.num_pages) { war_set_device_status(a.status_word, WAR_ERR_BAD_PAGE); pg = 0; }
                    const CUtensorMap* map = is_v ? &v_map : &k_map;
                    if (!kTokenMajor) {
                        if (stream_once) tma_load_block_hint(sRing + slot * kSlotBytes + lane * page_bytes, map, (int)(pg * a.Hkv + un.kvh), &bars->full[slot], evict_first);
                        else tma_load_block(sRing + slot * kSlotBytes + lane * page_bytes, map, (int)(pg * a.Hkv + un.kvh), &bars->full[slot]);
                    } else {
                        const uint32_t dst = sRing + slot * kSlotBytes + lane * (page_bytes >> 1);
                        tma_load_half_page(dst, map, 0, un.kvh, (int)pg, &bars->full[slot]);
                        tma_load_half_page(dst + 16384u, map, 64, un.kvh, (int)pg, &bars->full[slot]);
                    }
                }
                return true;
            };
            int pg_cur = page_of(0), pg_nxt = page_of(1);
            ok = load(0, pg_cur, false);                                    // K0
            for (int t = 0; t < T && ok; ++t) {
                const int pg_nn = page_of(t + 2);                            // page ids two tiles ahead, off the critical path
                if (t + 1 < T) ok = load(t + 1, pg_nxt, false);              // K(t+1)
                if (ok) ok = load(t, pg_cur, true);                          // V(t)
                pg_cur = pg_nxt; pg_nxt = pg_nn;
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------------ MMA issuer
        uint32_t ld0 = 0, cg[2] = {0, 0}, units_done = 0;
        constexpr uint32_t idesc_s = umma_idesc(128, 128, 0);
        constexpr uint32_t idesc_o = umma_idesc(128, 128, 1);
        constexpr uint32_t hi_q = umma_desc_hi(1024);
        const uint32_t q_lo = umma_desc_lo(sQ, 16);                  // Q: K-major, 8-row groups 1 KB apart
        // K: K-major; V: MN-major.  Head-major tiles: 8-row groups 2 KB apart, the 64-wide halves 1 KB apart.
        // Token-major tiles: 8-row groups 1 KB apart, the halves 16 KB apart.
        const uint32_t hi_kv = kTokenMajor ? umma_desc_hi(1024) : umma_desc_hi(2048);
        const uint32_t ring_lo = umma_desc_lo(sRing, 16);
        const uint32_t ring_lo_v = umma_desc_lo(sRing, kTokenMajor ? 16384 : 1024);
        const uint32_t k_half = (kTokenMajor ? 16384u : 1024u) >> 4;             // second 64 dims of K
        const uint32_t v_step = (kTokenMajor ? 2048u : 4096u) >> 4;              // 16 keys of V
        bool ok = true;
        fused_plan::Cursor cur{0, 0, 0};
        if (kFused) fused_plan::cursor_init(plan, cur);
        while (ok) {
            UnitView un;
            if (!fetch(cur, un)) break;
            const int T = un.tile_end - un.tile_begin;
            auto issue_s = [&](int t) -> bool {
                const uint32_t sq = seq_k(ld0, t), slot = sq % kSlots, g = t & 1;
                if (!mbar_wait(&bars->full[slot], (sq / kSlots) & 1u, bars, a.status_word)) return false;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t k_lo = ring_lo + slot * (kSlotBytes >> 4), d_s = tmem + g * 128u;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        constexpr uint32_t kHalfQ = 16384u >> 4;
                        const uint32_t qo = (uint32_t)(ks >> 2) * kHalfQ + (uint32_t)(ks & 3) * 2u;
                        const uint32_t ko = (uint32_t)(ks >> 2) * k_half + (uint32_t)(ks & 3) * 2u;
                        umma_bf16(d_s, pack64(q_lo + qo, hi_q), pack64(k_lo + ko, hi_kv), idesc_s, ks > 0);
                    }
                    umma_commit(&bars->s_ready[g]);
                    umma_commit(&bars->empty[slot]);
                }
                __syncwarp();
                return true;
            };
            ok = mbar_wait(&bars->q_ready, units_done & 1u, bars, a.status_word);
            if (ok) ok = issue_s(0);
            if (ok && T > 1) ok = issue_s(1);
            for (int t = 0; t < T && ok; ++t) {
                const uint32_t g = t & 1, tg = cg[g] + (uint32_t)(t >> 1);
                const uint32_t sq = seq_v(ld0, t, T), slot = sq % kSlots;
                const bool has_s = t + 2 < T;                        // S(t+2) goes out in the same burst as PV(t)
                const uint32_t sq_k = has_s ? seq_k(ld0, t + 2) : 0u, slot_k = sq_k % kSlots;
                ok = mbar_wait(&bars->p_ready[g], tg & 1u, bars, a.status_word) &&
                     mbar_wait(&bars->full[slot], (sq / kSlots) & 1u, bars, a.status_word);
                if (ok && has_s) ok = mbar_wait(&bars->full[slot_k], (sq_k / kSlots) & 1u, bars, a.status_word);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t v_lo = ring_lo_v + slot * (kSlotBytes >> 4), d_o = tmem + 256u + g * 128u, a_p = tmem + g * 128u;
                    const uint32_t acc0 = t > 1 ? 1u : 0u;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_bf16_ts(d_o, a_p + (uint32_t)ks * 8u, pack64(v_lo + (uint32_t)ks * v_step, hi_kv), idesc_o, ks > 0 ? 1u : acc0);
                    if (has_s) {
                        // sixteen MMAs back to back; the completion signals follow the burst (the one the softmax group
                        // waits for first)
                        const uint32_t k_lo = ring_lo + slot_k * (kSlotBytes >> 4), d_s = tmem + g * 128u;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            constexpr uint32_t kHalfQ = 16384u >> 4;
                            const uint32_t qo = (uint32_t)(ks >> 2) * kHalfQ + (uint32_t)(ks & 3) * 2u;
                            const uint32_t ko = (uint32_t)(ks >> 2) * k_half + (uint32_t)(ks & 3) * 2u;
                            umma_bf16(d_s, pack64(q_lo + qo, hi_q), pack64(k_lo + ko, hi_kv), idesc_s, ks > 0);
                        }
                        umma_commit(&bars->s_ready[g]);
                    }
                    umma_commit(&bars->pv_done[g]);
                    umma_commit(&bars->empty[slot]);
                    if (has_s) umma_commit(&bars->empty[slot_k]);
                }
                __syncwarp();
            }
            cg[0] += (uint32_t)(T + 1) >> 1;
            cg[1] += (uint32_t)T >> 1;
            ld0 += 2u * T;
            ++units_done;
        }
    } else if (kFused && warp == 10) {
        // ------------------------------------------------------------------ signaller (fused-plan variant)
        // Counts every split unit of this CTA whose partial result is out, for the CTA that merges the triple.  The
        // softmax warps only arrive on a barrier; the device-wide fence and the atomic sit here, off their path.
        uint32_t outs = 0;
        bool ok = true;
        fused_plan::Cursor cur{0, 0, 0};
        fused_plan::cursor_init(plan, cur);
        while (ok) {
            UnitView un;
            if (!fetch(cur, un)) break;
            if (un.n_chunks == 1) continue;
            const int32_t* prow = a.parent + (size_t)un.req * a.N;
            const int q0 = lane < a.N ? prow[lane] : 0, q1 = lane + 32 < a.N ? prow[lane + 32] : 0;
            if (tree_is_malformed(q0, q1, un.n_nodes, lane)) continue;          // (no partial is written for it)
            ok = mbar_wait(&bars->part_out, outs & 1u, bars, a.status_word);
            ++outs;
            if (ok && lane == 0) {
                __threadfence();
                count_arrival(&a.w.pair_count[(un.req * a.Hkv + un.kvh) * a.w.row_blocks + un.rb], a.call);
            }
            __syncwarp();
        }
    }
    } else {
        // ------------------------------------------------------------------ softmax groups, one thread per row
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        const int grp = warp >> 2;
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const uint32_t tS = tmem + grp * 128u + lane_addr;          // S, later P, of this group
        const uint32_t tO = tmem + 256u + grp * 128u + lane_addr;
        uint32_t ld0 = 0, cgm = 0, cg_other = 0, units_done = 0;    // cgm: tiles this group has processed so far
        bool ok = true;
        fused_plan::Cursor cur{0, 0, 0};
        if (kFused) fused_plan::cursor_init(plan, cur);
        while (ok) {
            UnitView un;
            if (!fetch(cur, un)) break;
            const int u = un.slot;
            const int i = un.req;
            const int n = un.n_nodes;
            const int R = a.G * n;
            const int pl = a.prefix_len[i];
            const int L = pl + n;
            const int gr = un.rb * kRowBlock + row;
            const bool in_tree = gr < R;
            const int j = in_tree ? gr / a.G : 0, g = in_tree ? gr % a.G : 0;
            const size_t qrow = ((size_t)i * a.N + j) * a.Hq + un.kvh * a.G + g;
            const int T = un.tile_end - un.tile_begin;
            // fused-plan variant: the plan has looked at num_nodes and prefix_len only; the tree itself is checked
            // below, by every warp that is about to use it (all come to the same verdict).  Its parent row is
            // requested here, ahead of the Q rows, and looked at after them.
            int q0 = 0, q1 = 0;
            if (kFused) {
                const int32_t* prow = a.parent + (size_t)i * a.N;
                q0 = lane < a.N ? prow[lane] : 0; q1 = lane + 32 < a.N ? prow[lane + 32] : 0;
            }
            // group 1 may not touch Q, O or its statistics before group 0 has finished the previous unit's epilogue
            if (grp == 1 && units_done > 0) {
                ok = mbar_wait(&bars->epi_done, (units_done - 1) & 1u, bars, a.status_word);
                if (!ok) break;
            }
            {   // each group writes one 64-wide half of every Q row (swizzled K-major)
                const uint4* src = reinterpret_cast<const uint4*>(a.q + qrow * 128) + grp * 8;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 x = in_tree ? src[c] : make_uint4(0, 0, 0, 0);
                    const uint32_t dst = sQ + (uint32_t)grp * 16384u + (uint32_t)row * 128u + (uint32_t)((c ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(x.x), "r"(x.y), "r"(x.z), "r"(x.w) : "memory");
                }
            }
            fence_async_proxy();
            mbar_arrive(&bars->q_ready);
            // A malformed tree makes its units run with no live row: nothing is written for the request.
            bool tree_ok = true;
            if (kFused) {
                tree_ok = !tree_is_malformed(q0, q1, n, lane);
                if (!tree_ok && lane == 0) war_set_device_status(a.status_word, WAR_ERR_BAD_TREE);
            }
            const bool valid = in_tree && tree_ok;
            const bool warp_valid = __any_sync(0xffffffffu, valid);
            uint64_t anc;
            if (kFused) {
                anc = tree_ok ? warp_ancestor_mask(q0, q1, n, j, lane) : 0ull;
                if (!valid) anc = 0ull;
            } else {
                anc = valid ? a.w.anc[(size_t)i * a.N + j] : 0ull;
            }
            float m_used = -CUDART_INF_F, l = 0.f;
            for (int t = grp; t < T && ok; t += 2, ++cgm) {
                const int key0 = (un.tile_begin + t) * kTileKeys;
                const bool need_mask = key0 + kTileKeys > pl;
                ok = mbar_wait(&bars->s_ready[grp], cgm & 1u, bars, a.status_word);
                if (!ok) break;
                tc_fence_after();
                if (warp_valid) {
                    // the whole row of S comes into registers once
                    uint32_t r[128];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, r + c * 32);
                    tmem_wait_ld();
                    if (need_mask) {
                        // Which of the tile's 128 keys this row sees, as a bit mask built once: the first d keys are
                        // prefix (all visible), key d + a is tree slot a (visible when a is the row's slot or an ancestor;
                        // the ancestor mask has no bit at or above num_nodes, so keys past the request's end are out).
                        // Two instructions per element afterwards: this path runs once per (request, kv head) and its
                        // code, fetched cold, competes with the main loop for the instruction cache.
                        const int d = pl - key0;                                  // < 128 here
                        unsigned long long lo, hi;
                        if (d >= 64) { lo = ~0ull; hi = ((1ull << (d - 64)) - 1ull) | (anc << (d - 64)); }
                        else if (d > 0) { lo = ((1ull << d) - 1ull) | (anc << d); hi = anc >> (64 - d); }
                        else { lo = d > -64 ? anc >> (-d) : 0ull; hi = 0ull; }
                        const uint32_t w[4] = {(uint32_t)lo, (uint32_t)(lo >> 32), (uint32_t)hi, (uint32_t)(hi >> 32)};
#pragma unroll
                        for (int e = 0; e < 128; ++e)
                            if (!((w[e >> 5] >> (e & 31)) & 1u)) r[e] = 0xff800000u;     // -inf
                    }
                    float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                    for (int e = 0; e < 128; e += 8) {                      // three-input max: two columns per instruction
#pragma unroll
                        for (int v = 0; v < 4; ++v) mx4[v] = max3(mx4[v], __uint_as_float(r[e + 2 * v]), __uint_as_float(r[e + 2 * v + 1]));
                    }
                    const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;    // scale > 0
                    float corr = 1.f;
                    bool rescale = false;
                    if (mx > m_used + kRescaleThreshold || (m_used == -CUDART_INF_F && mx > -CUDART_INF_F)) {
                        corr = exp2f(m_used - mx);                 // 0 when nothing was accumulated yet
                        l *= corr;
                        m_used = mx;
                        rescale = t > grp;                         // O of this group holds earlier tiles of the unit
                    }
                    const float neg_m = m_used == -CUDART_INF_F ? 0.f : -m_used;
                    // P = exp2(s*scale - m), packed to bf16 pairs in place (pair i lands in r[i], already consumed)
                    float2 l4[4] = {{0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}, {0.f, 0.f}};
                    const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nm2 = make_float2(neg_m, neg_m);
                    uint32_t* pk = r;
#pragma unroll
                    for (int e = 0; e < 128; e += 8) {
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            // two columns per FMA / add instruction (packed fp32 pairs)
                            const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[e + 2 * v]), __uint_as_float(r[e + 2 * v + 1])), sc2, nm2);
                            const float2 pp = make_float2(fast_exp2(x.x), fast_exp2(x.y));          // exp2(-inf) = 0
                            l4[v] = __fadd2_rn(l4[v], pp);
                            const __nv_bfloat162 h = __floats2bfloat162_rn(pp.x, pp.y);
                            pk[(e >> 1) + v] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                    }
                    l += ((l4[0].x + l4[0].y) + (l4[1].x + l4[1].y)) + ((l4[2].x + l4[2].y) + (l4[3].x + l4[3].y));
                    if (__any_sync(0xffffffffu, rescale)) {
                        // O of this group is stable once its previous P V product has completed
                        ok = mbar_wait(&bars->pv_done[grp], (cgm - 1) & 1u, bars, a.status_word);
                        ok = __all_sync(0xffffffffu, ok);
                        if (ok) {
                            tc_fence_after();
                            const float f = rescale ? corr : 1.f;
#pragma unroll 1                                                    // (rare: kept small, see the mask path above)
                            for (int c = 0; c < 4; ++c) {
                                uint32_t o[32];
                                tmem_ld32(tO + c * 32, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * f);
                                tmem_st32(tO + c * 32, o);
                            }
                        }
                    }
                    tmem_st32(tS, pk);
                    tmem_st32(tS + 32, pk + 32);
                    tmem_wait_st();
                }
                if (!ok) break;
                // the unit's last tile may hold rows past the request's last key: zero their V (P is exactly 0 there,
                // but 0 x NaN garbage would still poison the product)
                if (key0 + kTileKeys > L) {
                    const uint32_t sq = seq_v(ld0, t, T), slot = sq % kSlots;
                    ok = mbar_wait(&bars->full[slot], (sq / kSlots) & 1u, bars, a.status_word);
                    if (!ok) break;
                    if (row >= L - key0) {
                        const uint32_t base = sRing + slot * kSlotBytes +
                                              (kTokenMajor ? (uint32_t)row * 128u : (uint32_t)(row >> 3) * 2048u + (uint32_t)(row & 7) * 128u);
                        const uint32_t half = kTokenMajor ? 16384u : 1024u;
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int c = 0; c < 8; ++c)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(base + h * half + c * 16u), "r"(0) : "memory");
                    }
                    fence_async_proxy();
                }
                tc_fence_before();
                mbar_arrive(&bars->p_ready[grp]);
            }
            if (!ok) break;
            const uint32_t mine = (uint32_t)(T + 1 - grp) >> 1, theirs = (uint32_t)(T + grp) >> 1;   // tiles of this unit per group
            const bool fused_split = kFused && un.n_chunks != 1;
            if (grp == 1) {
                stats[row] = make_float2(m_used, l);
                mbar_arrive(&bars->stats_ready);
            } else {
                // epilogue: both groups' last products, then merge (max, sum, O) of the two groups and store
                ok = mbar_wait(&bars->pv_done[0], (cgm - 1) & 1u, bars, a.status_word) &&
                     mbar_wait(&bars->stats_ready, units_done & 1u, bars, a.status_word);
                if (ok && theirs > 0) ok = mbar_wait(&bars->pv_done[1], (cg_other + theirs - 1) & 1u, bars, a.status_word);
                if (!ok) break;
                tc_fence_after();
                if (warp_valid) {
                    const float2 st = stats[row];
                    const float m1 = theirs > 0 ? st.x : -CUDART_INF_F, l1 = theirs > 0 ? st.y : 0.f;
                    const float M = fmaxf(m_used, m1);
                    const float w0 = m_used == -CUDART_INF_F ? 0.f : exp2f(m_used - M);
                    const float w1 = m1 == -CUDART_INF_F ? 0.f : exp2f(m1 - M);
                    const float lsum = l * w0 + l1 * w1;
                    const bool split = un.n_chunks != 1;
                    const float f0 = split ? w0 : (lsum > 0.f ? w0 / lsum : 0.f), f1 = split ? w1 : (lsum > 0.f ? w1 / lsum : 0.f);
                    const bool use1 = theirs > 0;                  // uniform: O of group 1 is stale when it had no tile
#pragma unroll 1                                                    // (once per unit: kept small, see the mask path above)
                    for (int c = 0; c < 8; ++c) {
                        uint32_t o0[16], o1[16];
                        tmem_ld16(tO + c * 16, o0);
                        if (use1) tmem_ld16(tO + 128u + c * 16, o1);
                        tmem_wait_ld();
                        float x[16];
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            x[e] = __uint_as_float(o0[e]) * f0;
                            if (use1) x[e] = fmaf(__uint_as_float(o1[e]), f1, x[e]);
                        }
                        if (valid) {
                            if (!split) {
                                uint4* dst = reinterpret_cast<uint4*>(a.out + qrow * 128 + c * 16);
#pragma unroll
                                for (int v = 0; v < 2; ++v) {
                                    uint32_t w4[4];
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(x[v * 8 + 2 * e], x[v * 8 + 2 * e + 1]);
                                        w4[e] = *reinterpret_cast<const uint32_t*>(&h);
                                    }
                                    dst[v] = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                                }
                            } else {
                                float4* dst = reinterpret_cast<float4*>(a.w.part_o + ((size_t)u * a.w.rows + row) * 128 + c * 16);
#pragma unroll
                                for (int v = 0; v < 4; ++v) dst[v] = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
                            }
                        }
                    }
                    if (valid) {
                        if (!split) {
                            if (a.lse) a.lse[qrow] = (M + log2f(lsum)) * kLn2;
                        } else {
                            a.w.part_ml[((size_t)u * a.w.rows + row) * 2] = M;
                            a.w.part_ml[((size_t)u * a.w.rows + row) * 2 + 1] = lsum;
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive(&bars->epi_done);
                if (fused_split && tree_ok) mbar_arrive(&bars->part_out);     // this thread's share of the partial is written
            }
            (void)mine;
            cg_other += theirs;
            ld0 += 2u * T;
            ++units_done;
        }
        if (kFused && ok) {
            // ---- merges of split (request, kv head, row block) triples, by all eight softmax warps.  Contiguous
            // split: every CTA has at most one, the pair its last unit began.  Snake deal: the triples of all split
            // requests are dealt to the CTAs in turn, so the work at the end of the kernel is spread over all SMs.
            // Nothing waits for this CTA any more (its own partials are out), so waiting here cannot close a cycle. ----
            uint32_t merge_phase = 0;
            int share = kRowBlock;
            auto merge_one = [&](const UnitView& un, int part, int parts) -> bool {
                MergeArgs m;
                m.part = part; m.parts = parts; m.share = share;
                m.part_o = a.w.part_o; m.part_ml = a.w.part_ml; m.out = a.out; m.lse = a.lse; m.status_word = a.status_word;
                m.rows = a.w.rows; m.G = a.G; m.N = a.N; m.Hq = a.Hq;
                m.req = un.req; m.kvh = un.kvh; m.rb = un.rb; m.n_nodes = un.n_nodes; m.n_chunks = un.n_chunks;
                m.slot_base = un.slot_base; m.slot_stride = un.slot_stride; m.bump = un.bump;
                m.arrivals = &a.w.pair_count[(un.req * a.Hkv + un.kvh) * a.w.row_blocks + un.rb]; m.call = a.call;
                m.seen = &a.w.pair_seen[(un.req * a.Hkv + un.kvh) * a.w.row_blocks + un.rb];
                const bool done = merge_partials(m, smem, bars, &merge_phase);
                return done;
            };
            auto tree_bad = [&](int req, int n) -> bool {              // a malformed tree left no partials
                const int32_t* prow = a.parent + (size_t)req * a.N;
                const int q0 = lane < a.N ? prow[lane] : 0, q1 = lane + 32 < a.N ? prow[lane + 32] : 0;
                return tree_is_malformed(q0, q1, n, lane);
            };
            if (plan->mode == 1) {
                fused_plan::cursor_init(plan, cur);
                while (ok) {
                    UnitView un;
                    if (!fetch(cur, un)) break;
                    if (un.n_chunks == 1 || un.chunk != 0 || tree_bad(un.req, un.n_nodes)) continue;
                    ok = merge_one(un, 0, 1);
                }
            } else {
                // With few split triples every one is merged by two, four or eight CTAs, a share of its rows each: a
                // triple of many chunks is up to a megabyte that one SM would bring in and walk through in several
                // rounds.  Shares of at least 16 rows, on at most half of the CTAs (measured: 1 and 2 requests
                // with 128-row trees 74 -> 47 and 75 -> 64 us per call, 2 and 3 requests with 32-row trees 64 -> 60
                // and 71 -> 68; more shares than that bought nothing or cost a microsecond).
                const int n_split = plan->n_used, rows_blk = plan->t_all;
                int parts = 1, lg = 0;
                while (parts < 8 && 4 * parts * n_split <= (int)gridDim.x && rows_blk >= 32 * parts) { parts *= 2; ++lg; }
                share = (((rows_blk + parts - 1) >> lg) + 1) & ~1;
                int dealt = 0;                                         // shares of split requests before this one
#pragma unroll 1
                for (int p = 0; p < a.B && ok; ++p) {
                    const int i = plan->pos_req[p];
                    const int nc = plan->u.s.nc[i], n = plan->n[i];
                    if (nc <= 1 || n == 0) continue;
                    const int rbs = (a.G * n + kRowBlock - 1) / kRowBlock, per = a.Hkv * rbs, shares = per * parts;
                    int k = ((int)blockIdx.x - dealt) % (int)gridDim.x;
                    if (k < 0) k += gridDim.x;
                    dealt += shares;
                    if (k >= shares || tree_bad(i, n)) continue;
#pragma unroll 1
                    for (; k < shares && ok; k += gridDim.x) {
                        const int part = k / per, tr = k - part * per;       // the shares of a triple sit `per` CTAs apart
                        UnitView un;
                        un.req = i; un.kvh = tr / rbs; un.rb = tr - un.kvh * rbs; un.n_nodes = n; un.n_chunks = nc; un.chunk = 0;
                        un.tile_begin = un.tile_end = 0; un.slot = 0;
                        un.slot_base = (int)plan->u.s.pos_base[p] + tr; un.slot_stride = per; un.bump = 0;
                        ok = merge_one(un, part, parts);
                    }
                }
            }
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

// A head-major pool [num_pages, Hkv, page_size, 128] bf16 seen as blocks of (page, head): [blocks][token/8][d/64][token%8][d%64].
// A token-major pool (page, token, head, d) seen as (d, token, head, page) with a box of 64 dims x all tokens of one head.
bool make_pool_map(CUtensorMap* map, const void* pool, long long num_pages, int Hkv, int page_size, int token_major) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    if (token_major) {
        const cuuint64_t dims[4] = {128, (cuuint64_t)page_size, (cuuint64_t)Hkv, (cuuint64_t)num_pages};
        const cuuint64_t strides[3] = {(cuuint64_t)Hkv * 256, 256, (cuuint64_t)page_size * Hkv * 256};
        const cuuint32_t box[4] = {64, (cuuint32_t)page_size, 1, 1};
        return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    }
    const cuuint64_t dims[5] = {64, 8, 2, (cuuint64_t)(page_size / 8), (cuuint64_t)(num_pages * Hkv)};
    const cuuint64_t strides[4] = {256, 128, 2048, (cuuint64_t)page_size * 256};
    const cuuint32_t box[5] = {64, 8, 2, (cuuint32_t)(page_size / 8), 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(pool), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The two tensor maps of a call depend only on the pools (address, pages, heads, page size, layout), which an engine
// keeps for its whole life, so they are encoded once and looked up afterwards: a handful of entries, most recent first.
struct PoolMapKey {
    const void* k; const void* v; long long num_pages; int Hkv, page_size, token_major, dev;
    bool operator==(const PoolMapKey& o) const {
        return k == o.k && v == o.v && num_pages == o.num_pages && Hkv == o.Hkv && page_size == o.page_size &&
               token_major == o.token_major && dev == o.dev;
    }
};
struct PoolMaps { PoolMapKey key; CUtensorMap k_map, v_map; bool used; };
constexpr int kMapCacheEntries = 8;
std::mutex g_map_lock;
PoolMaps g_map_cache[kMapCacheEntries];

bool pool_maps(const PoolMapKey& key, CUtensorMap* k_map, CUtensorMap* v_map) {
    std::lock_guard<std::mutex> g(g_map_lock);
    for (int e = 0; e < kMapCacheEntries; ++e) {
        if (g_map_cache[e].used && g_map_cache[e].key == key) {
            const PoolMaps hit = g_map_cache[e];
            for (int m = e; m > 0; --m) g_map_cache[m] = g_map_cache[m - 1];
            g_map_cache[0] = hit;
            *k_map = hit.k_map; *v_map = hit.v_map;
            return true;
        }
    }
    PoolMaps fresh;
    fresh.key = key; fresh.used = true;
    if (!make_pool_map(&fresh.k_map, key.k, key.num_pages, key.Hkv, key.page_size, key.token_major) ||
        !make_pool_map(&fresh.v_map, key.v, key.num_pages, key.Hkv, key.page_size, key.token_major))
        return false;
    for (int m = kMapCacheEntries - 1; m > 0; --m) g_map_cache[m] = g_map_cache[m - 1];
    g_map_cache[0] = fresh;
    *k_map = fresh.k_map; *v_map = fresh.v_map;
    return true;
}

// Call numbers of the one-launch path: 48 bits, never 0, no two launches of this process alike (the start is taken
// from the clock so that a word left by an earlier process does not look current either).
unsigned long long next_call_number() {
    static std::atomic<unsigned long long> counter{
        (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() * 0x9E3779B97F4A7C15ull};
    unsigned long long v;
    do { v = counter.fetch_add(1) & 0xFFFFFFFFFFFFull; } while (v == 0);
    return v;
}

// Per-device set-up (SM count, shared-memory opt-in of the four kernel variants), once per device.
constexpr int kMaxDevices = 64;
std::once_flag g_dev_once[kMaxDevices];
int g_sm_count[kMaxDevices];
war_status_t g_dev_status[kMaxDevices];

war_status_t device_setup(int dev) {
    std::call_once(g_dev_once[dev], [dev]() {
        g_dev_status[dev] = WAR_ERR_CUDA;
        if (cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
        if (cudaFuncSetAttribute(attn_sm100_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return;
        if (cudaFuncSetAttribute(attn_sm100_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return;
        if (cudaFuncSetAttribute(attn_sm100_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytesFused) != cudaSuccess) return;
        if (cudaFuncSetAttribute(attn_sm100_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytesFused) != cudaSuccess) return;
        g_dev_status[dev] = WAR_OK;
    });
    if (g_dev_status[dev] != WAR_OK) (void)cudaGetLastError();
    return g_dev_status[dev];
}

}  // namespace

namespace {
// Self-test of the bounded waits (see war.h): one CTA, an mbarrier nobody ever arrives on.  Warp 0 waits on it with
// the caller's budget through the same mbar_wait the attention kernel uses, runs out of it, records WAR_ERR_TIMEOUT
// and raises the abort flag; warp 1 waits on the same barrier with the kernel's ordinary (long) budget and is
// released by that flag.  result = { warp 0's wait returned true?, warp 1's, ns warp 0 waited, ns warp 1 waited }.
struct SelftestBars { uint64_t never; int abort_flag; };
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(unsigned long long budget_ns, long long* result, int* status_word) {
    __shared__ SelftestBars bars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&bars.never, 1);
        bars.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const unsigned long long t0 = global_timer_ns();
    const bool ok = warp == 0 ? mbar_wait(&bars.never, 0u, &bars, status_word, budget_ns)
                              : mbar_wait(&bars.never, 0u, &bars, status_word);
    const unsigned long long dt = global_timer_ns() - t0;
    if (lane == 0) { result[warp] = ok ? 1 : 0; result[2 + warp] = (long long)dt; }
}

}  // namespace

extern "C" war_status_t war_selftest_bounded_wait(int32_t budget_us, int64_t* d_result, war_stream_t stream) {
    if (!d_result || budget_us < 1 || budget_us > 1000000) return WAR_ERR_INVALID_ARG;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>((unsigned long long)budget_us * 1000ull, (long long*)d_result, status_word);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}

int war_attn_sm_count() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return 0; }
    return device_setup(dev) == WAR_OK ? g_sm_count[dev] : 0;
}

war_status_t war_attn_launch_sm100(const void* q, const void* k, const void* v, const int32_t* page_table,
                                   const int32_t* prefix_len, const int32_t* num_nodes, const int32_t* parent,
                                   const war_attn_params_t* p, const AttnWorkspace& w, bool fused,
                                   void* out, float* lse, int* status_word, cudaStream_t s) {
    int dev = 0;
    WAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return WAR_ERR_UNSUPPORTED;
    const war_status_t st = device_setup(dev);
    if (st != WAR_OK) return st;
    if (p->num_pages == 0) return WAR_ERR_INVALID_ARG;
    CUtensorMap k_map, v_map;
    const int token_major = war_attn_pool_layout(p->k_strides, p) == 1;
    const PoolMapKey key{k, v, p->num_pages, p->Hkv, p->page_size, token_major, dev};
    if (!pool_maps(key, &k_map, &v_map)) return WAR_ERR_CUDA;
    KernelArgs a;
    a.q = (const __nv_bfloat16*)q; a.page_table = page_table; a.prefix_len = prefix_len;
    a.out = (__nv_bfloat16*)out; a.lse = lse; a.status_word = status_word; a.w = w;
    a.num_pages = p->num_pages; a.scale_log2 = p->scale * kLog2e;
    a.N = p->N; a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv; a.page_size = p->page_size; a.max_pages = p->max_pages_per_req;
    a.num_nodes = num_nodes; a.parent = parent; a.B = p->B; a.call = 0;
    const int grid = g_sm_count[dev];
    if (fused) {
        a.call = next_call_number();
        if (token_major) attn_sm100_kernel<true, true><<<grid, kThreads, kSmemBytesFused, s>>>(k_map, v_map, a);
        else attn_sm100_kernel<false, true><<<grid, kThreads, kSmemBytesFused, s>>>(k_map, v_map, a);
    } else {
        if (token_major) attn_sm100_kernel<true, false><<<grid, kThreads, kSmemBytes, s>>>(k_map, v_map, a);
        else attn_sm100_kernel<false, false><<<grid, kThreads, kSmemBytes, s>>>(k_map, v_map, a);
    }
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
