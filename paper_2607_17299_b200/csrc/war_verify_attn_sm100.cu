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
#include <cuda.h>
#include <cuda_bf16.h>
#include <math_constants.h>
#include "war_common.cuh"
#include "war_attn_plan.cuh"
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
constexpr int kSmemBytes = kOffStats + 1024 + 1024;

struct Bars {
    uint64_t full[kSlots], empty[kSlots];
    uint64_t s_ready[2], p_ready[2], pv_done[2];
    uint64_t q_ready, stats_ready, epi_done;
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
};

template <bool kTokenMajor>                         // pool layout: false = (page, head, token, d), true = (page, token, head, d)
__global__ void __launch_bounds__(kThreads, 1)
attn_sm100_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const KernelArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    Bars* bars = (Bars*)(smem + kOffBar);
    float2* stats = (float2*)(smem + kOffStats);     // group 1's (max, sum) per row, for the merge
    const uint32_t sQ = smem_u32(smem + kOffQ), sRing = smem_u32(smem + kOffRing);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_units = a.w.counters[1];
    // k-th unit of this CTA: its own contiguous list, or the snake deal of the longest-first list
    const bool contiguous = a.w.counters[3] != 0 && gridDim.x <= (unsigned)kMaxPlanCtas;
    const int list_first = contiguous ? a.w.cta_first[blockIdx.x] : 0, list_end = contiguous ? a.w.cta_first[blockIdx.x + 1] : 0;
    auto unit_at = [&](int k) -> int {
        if (contiguous) return list_first + k < list_end ? list_first + k : n_units;
        return snake_unit(k, blockIdx.x, gridDim.x);
    };
    const int pages_per_tile = kTileKeys / a.page_size;
    const uint32_t page_bytes = (uint32_t)a.page_size * 256u;

    if (tid == 0) {
        for (int i = 0; i < kSlots; ++i) { mbar_init(&bars->full[i], 1); mbar_init(&bars->empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&bars->s_ready[i], 1); mbar_init(&bars->p_ready[i], 128); mbar_init(&bars->pv_done[i], 1); }
        mbar_init(&bars->q_ready, 256);
        mbar_init(&bars->stats_ready, 128);
        mbar_init(&bars->epi_done, 128);
        bars->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
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
        uint32_t ld = 0;
        bool ok = true;
        for (int k = 0; ok; ++k) {
            const int u = unit_at(k);
            if (u >= n_units) break;
            const AttnUnit un = a.w.units[u];
            const int i = un.req;
            const int L = a.prefix_len[i] + a.w.req[i].n_nodes;
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
                        tma_load_block(sRing + slot * kSlotBytes + lane * page_bytes, map, (int)(pg * a.Hkv + un.kvh), &bars->full[slot]);
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
        for (int k = 0; ok; ++k) {
            const int u = unit_at(k);
            if (u >= n_units) break;
            const AttnUnit un = a.w.units[u];
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
        for (int k = 0; ok; ++k) {
            const int u = unit_at(k);
            if (u >= n_units) break;
            const AttnUnit un = a.w.units[u];
            const int i = un.req;
            const int n = a.w.req[i].n_nodes;
            const int R = a.G * n;
            const int pl = a.prefix_len[i];
            const int L = pl + n;
            const int gr = un.rb * kRowBlock + row;
            const bool valid = gr < R;
            const bool warp_valid = __any_sync(0xffffffffu, valid);
            const int j = valid ? gr / a.G : 0, g = valid ? gr % a.G : 0;
            const size_t qrow = ((size_t)i * a.N + j) * a.Hq + un.kvh * a.G + g;
            const uint64_t anc = valid ? a.w.anc[(size_t)i * a.N + j] : 0ull;
            const int T = un.tile_end - un.tile_begin;
            // group 1 may not touch Q, O or its statistics before group 0 has finished the previous unit's epilogue
            if (grp == 1 && units_done > 0) {
                ok = mbar_wait(&bars->epi_done, (units_done - 1) & 1u, bars, a.status_word);
                if (!ok) break;
            }
            {   // each group writes one 64-wide half of every Q row (swizzled K-major)
                const uint4* src = reinterpret_cast<const uint4*>(a.q + qrow * 128) + grp * 8;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const uint4 x = valid ? src[c] : make_uint4(0, 0, 0, 0);
                    const uint32_t dst = sQ + (uint32_t)grp * 16384u + (uint32_t)row * 128u + (uint32_t)((c ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(x.x), "r"(x.y), "r"(x.z), "r"(x.w) : "memory");
                }
            }
            fence_async_proxy();
            mbar_arrive(&bars->q_ready);
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
#pragma unroll
                        for (int e = 0; e < 128; ++e)
                            if (!key_visible(key0 + e, pl, L, anc)) r[e] = 0xff800000u;     // -inf
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
#pragma unroll
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
#pragma unroll
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
            }
            (void)mine;
            cg_other += theirs;
            ld0 += 2u * T;
            ++units_done;
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

}  // namespace

war_status_t war_attn_launch_sm100(const void* q, const void* k, const void* v, const int32_t* page_table,
                                   const int32_t* prefix_len, const war_attn_params_t* p, const AttnWorkspace& w,
                                   void* out, float* lse, int* status_word, cudaStream_t s) {
    static int sm_count[64] = {0};
    static bool attr_set[64] = {false};
    int dev = 0;
    WAR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return WAR_ERR_UNSUPPORTED;
    if (!sm_count[dev]) WAR_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    if (!attr_set[dev]) {
        WAR_CUDA_TRY(cudaFuncSetAttribute(attn_sm100_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        WAR_CUDA_TRY(cudaFuncSetAttribute(attn_sm100_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        attr_set[dev] = true;
    }
    if (p->num_pages == 0) return WAR_ERR_INVALID_ARG;
    CUtensorMap k_map, v_map;
    const int token_major = war_attn_pool_layout(p->k_strides, p) == 1;
    if (!make_pool_map(&k_map, k, p->num_pages, p->Hkv, p->page_size, token_major) ||
        !make_pool_map(&v_map, v, p->num_pages, p->Hkv, p->page_size, token_major))
        return WAR_ERR_CUDA;
    KernelArgs a;
    a.q = (const __nv_bfloat16*)q; a.page_table = page_table; a.prefix_len = prefix_len;
    a.out = (__nv_bfloat16*)out; a.lse = lse; a.status_word = status_word; a.w = w;
    a.num_pages = p->num_pages; a.scale_log2 = p->scale * kLog2e;
    a.N = p->N; a.Hq = p->Hq; a.Hkv = p->Hkv; a.G = p->Hq / p->Hkv; a.page_size = p->page_size; a.max_pages = p->max_pages_per_req;
    if (token_major) attn_sm100_kernel<true><<<sm_count[dev], kThreads, kSmemBytes, s>>>(k_map, v_map, a);
    else attn_sm100_kernel<false><<<sm_count[dev], kThreads, kSmemBytes, s>>>(k_map, v_map, a);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
