// war_draft_local: draft trees from each request's own context, and war_draft_pick: the choice between two trees.
//
// The SuffixDecoding method that the paper adopts (Section 3.3) also drafts from the tokens of the running request
// itself: text a rollout has produced or read once tends to come back inside the same trajectory.  A context changes
// every step, so no index is kept for it: a cluster of up to 8 CTAs per request scans the context, a slice each (4
// bytes per token, a few microseconds even at 10^5 tokens), for the longest suffix that occurs earlier and for its 32
// most recent occurrences; the slices' results meet in the first CTA's shared memory (distributed shared memory and
// the hardware cluster barrier: no flags, no spinning).  Warp 0 of that CTA builds the tree with one occurrence per
// lane: a node is a lane mask plus a depth, its continuations are the groups of equal next tokens
// (`__match_any_sync`), and offers are taken best-first exactly as in war_draft.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include "war.h"
#include "war_common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxN = 64;
constexpr int kMaxK = 8;
constexpr int kMaxP = 32;
constexpr int kMaxOcc = 32;                   // occurrences used per request: the most recent ones
constexpr int kScanDepth = 8;                 // positions per thread and scan step, all loads in flight together
constexpr int kChunk = kThreads * kScanDepth;

struct Shared {
    int pat[kMaxP];                           // pat[t] = token t places before the end of the context
    int best_len, n_occ, n_running, stop;
    unsigned chunk_mask[kScanDepth][kWarps];
    int occ[kMaxOcc];                         // end positions of the occurrences used, most recent first
    // offers: the rank-r continuation of slot j sits at j * kMaxK + r, in the order (count desc, token asc); count 0
    // ends a slot's list
    int pool_cnt[kMaxN * kMaxK], pool_tok[kMaxN * kMaxK];
    unsigned pool_mask[kMaxN * kMaxK];
    int slot_depth[kMaxN];
    unsigned slot_mask[kMaxN];
};

__global__ void __launch_bounds__(kThreads)
war_draft_local_kernel(const int32_t* __restrict__ ctx, const int64_t* __restrict__ ctx_off, const int32_t* __restrict__ tail_len,
                       int B, int P, int N, int K, int min_match, int spec_batch_limit, int fac_num, int fac_den, int prob_num,
                       int prob_den, int32_t* __restrict__ match_len, int32_t* __restrict__ num_nodes, int32_t* __restrict__ ids,
                       int32_t* __restrict__ parent, int32_t* __restrict__ count, int* status_word) {
    __shared__ Shared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank(), nblk = (int)cluster.num_blocks();      // the CTAs of a cluster share a request
    const int b = blockIdx.x / nblk;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int32_t* o_ids = ids + (size_t)b * N;
    int32_t* o_par = parent + (size_t)b * N;
    int32_t* o_cnt = count ? count + (size_t)b * N : nullptr;

    // workload-aware switch, as in war_draft: every CTA counts the running requests itself
    bool plain = false;
    if (tid == 0) { sh.n_running = 0; sh.best_len = 0; sh.n_occ = 0; sh.stop = 0; }
    cluster.sync();                                                       // before any CTA touches another one's shared memory
    if (spec_batch_limit > 0) {
        int c = 0;
        for (int i = tid; i < B; i += kThreads) c += tail_len[i] >= 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0 && c) atomicAdd(&sh.n_running, c);
        __syncthreads();
        plain = sh.n_running > spec_batch_limit;
    }
    const int my_tl = tail_len[b];
    const long long len64 = ctx_off[b + 1] - ctx_off[b];
    const bool bad = len64 < 0 || len64 > 0x7fffffffll;
    if (bad && tid == 0) war_set_device_status(status_word, WAR_ERR_INVALID_ARG);
    const int L = bad ? 0 : (int)len64;
    const int32_t* c = ctx + ctx_off[b];

    auto finish = [&](int ml, int n) {                                   // all threads: lengths, then the unused slots
        if (rank != 0) return;                                           // (every early exit is taken by the whole cluster)
        if (tid == 0) { match_len[b] = ml; num_nodes[b] = n; }
        for (int j = n + tid; j < N; j += kThreads) {
            o_ids[j] = -1; o_par[j] = -1;
            if (o_cnt) o_cnt[j] = 0;
        }
    };
    if (my_tl < 0 || bad) { finish(0, 0); return; }
    if (tid == 0 && rank == 0) { o_ids[0] = L > 0 ? c[L - 1] : -1; o_par[0] = -1; if (o_cnt) o_cnt[0] = 0; }
    int maxlen = min(min(P, my_tl), L - 1);
    if (plain || maxlen <= 0) { finish(0, 1); return; }

    // the pattern, last token first; a token < 0 never matches, so the pattern ends before it
    if (tid < maxlen) sh.pat[tid] = c[L - 1 - tid];
    __syncthreads();
    {
        int first_neg = maxlen;
        for (int t = 0; t < maxlen; ++t) if (sh.pat[t] < 0) { first_neg = t; break; }
        maxlen = first_neg;                                               // the same in every thread
    }
    if (maxlen == 0) { finish(0, 1); return; }

    // this CTA's slice of the end positions 0 .. L - 2
    const int slice = (L - 1 + nblk - 1) / nblk;
    const int s_lo = min(rank * slice, L - 1), s_hi = min(s_lo + slice, L - 1);
    // ---- pass 1: the longest suffix that also ends at some position e <= L - 2 ----
    // (kScanDepth coalesced loads per thread are in flight together: a CTA alone has to cover the latency)
    {
        const int last = sh.pat[0];
        int best = 0;
        for (int base = s_lo; base < s_hi; base += kChunk) {
            int v[kScanDepth];
#pragma unroll
            for (int k = 0; k < kScanDepth; ++k) {
                const int e = base + k * kThreads + tid;
                v[k] = e < s_hi ? c[e] : -1;
            }
#pragma unroll
            for (int k = 0; k < kScanDepth; ++k) {
                if (v[k] != last) continue;
                const int e = base + k * kThreads + tid;
                const int lim = min(maxlen, e + 1);
                int m = 1;
                while (m < lim && c[e - m] == sh.pat[m]) ++m;
                best = max(best, m);
            }
        }
        best = __reduce_max_sync(0xffffffffu, best);
        if (lane == 0 && best > 0) atomicMax(cluster.map_shared_rank(&sh.best_len, 0), best);     // the first CTA collects
    }
    cluster.sync();
    const int ml = *cluster.map_shared_rank(&sh.best_len, 0);
    if (ml == 0) { cluster.sync(); finish(0, 1); return; }             // (nobody leaves while its memory may be read)

    // ---- pass 2: its most recent occurrences, kChunk positions at a time from the end of the context ----
    for (int hi = s_hi; hi > s_lo; hi -= kChunk) {                        // positions [max(hi - kChunk, s_lo), hi)
        int v[kScanDepth];
#pragma unroll
        for (int k = 0; k < kScanDepth; ++k) {
            const int e = hi - kChunk + k * kThreads + tid;
            v[k] = e >= max(ml - 1, s_lo) ? c[e] : -1;
        }
        unsigned hits = 0;
#pragma unroll
        for (int k = 0; k < kScanDepth; ++k) {
            const int e = hi - kChunk + k * kThreads + tid;
            bool hit = v[k] == sh.pat[0];                                 // (a pattern token is never negative)
            for (int t = 1; hit && t < ml; ++t) hit = c[e - t] == sh.pat[t];
            hits |= (unsigned)hit << k;
        }
        if (__syncthreads_count(hits != 0) == 0) continue;               // nothing in this chunk (the usual case)
#pragma unroll
        for (int k = 0; k < kScanDepth; ++k) {
            const unsigned m = __ballot_sync(0xffffffffu, (hits >> k) & 1u);
            if (lane == 0) sh.chunk_mask[k][warp] = m;
        }
        __syncthreads();
        if (tid == 0) {
            int n = sh.n_occ;
            for (int k = kScanDepth - 1; k >= 0 && n < kMaxOcc; --k)
                for (int w = kWarps - 1; w >= 0 && n < kMaxOcc; --w) {
                    unsigned x = sh.chunk_mask[k][w];
                    while (x && n < kMaxOcc) {
                        const int bit = 31 - __clz(x);
                        sh.occ[n++] = hi - kChunk + k * kThreads + w * 32 + bit;
                        x &= ~(1u << bit);
                    }
                }
            sh.n_occ = n;
            sh.stop = n >= kMaxOcc;
        }
        __syncthreads();
        if (sh.stop) break;
    }
    // the slices' lists meet in the first CTA, most recent slice first
    cluster.sync();
    if (rank == 0 && warp == 0 && nblk > 1) {
        int have = 0, mine = 0;
        for (int r = nblk - 1; r >= 0 && have < kMaxOcc; --r) {
            const int n_r = min(*cluster.map_shared_rank(&sh.n_occ, r), kMaxOcc - have);
            if (lane >= have && lane < have + n_r) mine = cluster.map_shared_rank(sh.occ, r)[lane - have];
            have += n_r;
        }
        __syncwarp();
        if (lane < have) sh.occ[lane] = mine;
        if (lane == 0) sh.n_occ = have;
    }
    cluster.sync();                                                       // the other CTAs' lists have been read
    if (rank != 0) return;
    __syncthreads();
    const int n_occ = sh.n_occ;                                           // >= 1: pass 1 saw one

    // ---- the tree: warp 0, one occurrence per lane ----
    if (warp == 0) {
        const int e = lane < n_occ ? sh.occ[lane] : 0;
        const int n_cap = fac_num > 0 ? min(N, 1 + (int)(((long long)ml * fac_num) / fac_den)) : N;
        int n_nodes = 1, head0 = 0, head1 = 0, cur0 = 0, cur1 = 0;         // offer lists of slots lane and lane + 32
        if (lane == 0) {
            if (o_cnt) o_cnt[0] = n_occ;
            sh.slot_depth[0] = 0;
            sh.slot_mask[0] = n_occ >= 32 ? 0xffffffffu : ((1u << n_occ) - 1u);
        }
        __syncwarp();
        int slot = ml >= max(1, min_match) && n_cap > 1 ? 0 : -1;          // the slot to expand next
        while (slot >= 0) {
            // continuations of this slot: groups of equal next tokens among its occurrences
            const int d = sh.slot_depth[slot];
            const unsigned mask = sh.slot_mask[slot];
            const int pos = e + d + 1;
            const int t = ((mask >> lane) & 1u) && pos <= L - 1 ? c[pos] : -1;
            const bool valid = t >= 0;
            const unsigned gm = __match_any_sync(0xffffffffu, valid ? t : -1 - lane);
            const int cnt = __popc(gm);
            bool head = valid && lane == __ffs(gm) - 1;
            const int parent_cnt = __popc(mask);
            int n_fin = 0;
            for (int r = 0; r < K; ++r) {
                const int c_best = __reduce_max_sync(0xffffffffu, head ? cnt : 0);
                if (c_best == 0) break;
                const int t_best = __reduce_min_sync(0xffffffffu, head && cnt == c_best ? t : 0x7fffffff);
                if (head && cnt == c_best && t == t_best) {              // one lane: this group is the slot's rank-r offer
                    const bool keep = prob_num == 0 || (long long)cnt * prob_den >= (long long)prob_num * parent_cnt;
                    const int at = slot * kMaxK + r;
                    sh.pool_cnt[at] = keep ? cnt : 0; sh.pool_tok[at] = t; sh.pool_mask[at] = gm;
                    head = false;
                }
                __syncwarp();
                ++n_fin;
            }
            if (lane >= n_fin && lane < kMaxK) sh.pool_cnt[slot * kMaxK + lane] = 0;
            __syncwarp();
            if (lane == (slot & 31)) {                                    // the list's owner picks up its head
                const int h = sh.pool_cnt[slot * kMaxK];
                if (slot < 32) { head0 = h; cur0 = 0; } else { head1 = h; cur1 = 0; }
            }
            __syncwarp();
            // best offer of all lists: count desc, parent slot asc, token asc (= rank asc within a list)
            const int c_best = __reduce_max_sync(0xffffffffu, max(head0, head1));
            if (c_best <= 0) break;
            const int mine = head0 == c_best ? (lane * kMaxK + cur0) : head1 == c_best ? ((lane + 32) * kMaxK + cur1) : 0x7fffffff;
            const int bi = __reduce_min_sync(0xffffffffu, mine);
            const int bp = bi / kMaxK, j = n_nodes;
            if (lane == (bp & 31)) {
                o_ids[j] = sh.pool_tok[bi]; o_par[j] = bp;
                if (o_cnt) o_cnt[j] = c_best;
                sh.slot_depth[j] = sh.slot_depth[bp] + 1;
                sh.slot_mask[j] = sh.pool_mask[bi];
                const int nr = (bi & (kMaxK - 1)) + 1;
                const int nh = nr < kMaxK ? sh.pool_cnt[bi + 1] : 0;
                if (bp < 32) { cur0 = nr; head0 = nh; } else { cur1 = nr; head1 = nh; }
            }
            __syncwarp();
            ++n_nodes;
            slot = n_nodes < n_cap ? j : -1;                              // the last slot of the budget is not expanded
        }
        if (lane == 0) sh.n_occ = n_nodes;                                // hand the slot count to the whole CTA
    }
    __syncthreads();
    finish(ml, sh.n_occ);
}

// a / b > c / d for non-negative numerators below 2^63 and positive denominators (128-bit products)
__device__ __forceinline__ bool frac_greater(unsigned long long a, unsigned long long b, unsigned long long c, unsigned long long d) {
    const unsigned long long l_hi = __umul64hi(a, d), l_lo = a * d, r_hi = __umul64hi(c, b), r_lo = c * b;
    return l_hi > r_hi || (l_hi == r_hi && l_lo > r_lo);
}

// One warp per request: score = (sum of count[1 .. n)) / count[0] of each tree; the second tree wins only with a
// strictly larger score.
__global__ void __launch_bounds__(256)
war_draft_pick_kernel(int B, int N, const int32_t* __restrict__ a_ml, const int32_t* __restrict__ a_nn, const int32_t* __restrict__ a_ids,
                      const int32_t* __restrict__ a_par, const int32_t* __restrict__ a_cnt, const int32_t* __restrict__ b_ml,
                      const int32_t* __restrict__ b_nn, const int32_t* __restrict__ b_ids, const int32_t* __restrict__ b_par,
                      const int32_t* __restrict__ b_cnt, int32_t* __restrict__ source, int32_t* __restrict__ o_ml,
                      int32_t* __restrict__ o_nn, int32_t* __restrict__ o_ids, int32_t* __restrict__ o_par, int32_t* __restrict__ o_cnt) {
    const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (i >= B) return;
    const int na = min(max(a_nn[i], 0), N), nb = min(max(b_nn[i], 0), N);
    unsigned long long sa = 0, sb = 0;
    for (int j = 1 + lane; j < na; j += 32) sa += (unsigned)max(a_cnt[(size_t)i * N + j], 0);
    for (int j = 1 + lane; j < nb; j += 32) sb += (unsigned)max(b_cnt[(size_t)i * N + j], 0);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { sa += __shfl_xor_sync(0xffffffffu, sa, o); sb += __shfl_xor_sync(0xffffffffu, sb, o); }
    const unsigned long long da = na > 0 ? (unsigned)max(a_cnt[(size_t)i * N], 0) : 0, db = nb > 0 ? (unsigned)max(b_cnt[(size_t)i * N], 0) : 0;
    if (da == 0) sa = 0;                                                  // no occurrences: score 0
    if (db == 0) sb = 0;
    const bool second = frac_greater(sb, db ? db : 1, sa, da ? da : 1);
    const int32_t* s_ids = second ? b_ids : a_ids;
    const int32_t* s_par = second ? b_par : a_par;
    const int32_t* s_cnt = second ? b_cnt : a_cnt;
    if (lane == 0) { source[i] = second; o_ml[i] = second ? b_ml[i] : a_ml[i]; o_nn[i] = second ? b_nn[i] : a_nn[i]; }
    for (int j = lane; j < N; j += 32) {
        o_ids[(size_t)i * N + j] = s_ids[(size_t)i * N + j];
        o_par[(size_t)i * N + j] = s_par[(size_t)i * N + j];
        if (o_cnt) o_cnt[(size_t)i * N + j] = s_cnt[(size_t)i * N + j];
    }
}

}  // namespace

extern "C" war_status_t war_draft_local(const int32_t* d_ctx, const int64_t* d_ctx_off, const int32_t* d_tail_len,
                                        const war_draft_params_t* p, int32_t* d_match_len, int32_t* d_num_nodes,
                                        int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream) {
    if (!p) return WAR_ERR_INVALID_ARG;
    if (p->B < 0 || p->P < 1 || p->P > kMaxP || p->N < 1 || p->N > kMaxN || p->topk < 1 || p->topk > kMaxK || p->min_match < 0 ||
        p->spec_batch_limit < 0 || p->spec_factor_num < 0 || (p->spec_factor_num > 0 && p->spec_factor_den < 1) ||
        p->min_prob_num < 0 || (p->min_prob_num > 0 && (p->min_prob_den < 1 || p->min_prob_num > p->min_prob_den)))
        return WAR_ERR_INVALID_ARG;
    if (p->B == 0) return WAR_OK;
    if (!d_ctx || !d_ctx_off || !d_tail_len || !d_match_len || !d_num_nodes || !d_ids || !d_parent) return WAR_ERR_INVALID_ARG;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    // CTAs per request: as many as still leave the whole grid a few waves at most
    const int nblk = p->B <= 128 ? 8 : p->B <= 256 ? 4 : p->B <= 512 ? 2 : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p->B * nblk);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = nblk; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int fac_den = p->spec_factor_num > 0 ? p->spec_factor_den : 1, prob_den = p->min_prob_num > 0 ? p->min_prob_den : 1;
    WAR_CUDA_TRY(cudaLaunchKernelEx(&cfg, war_draft_local_kernel, d_ctx, d_ctx_off, d_tail_len, (int)p->B, (int)p->P, (int)p->N,
                                    (int)p->topk, (int)p->min_match, (int)p->spec_batch_limit, (int)p->spec_factor_num, fac_den,
                                    (int)p->min_prob_num, prob_den, d_match_len, d_num_nodes, d_ids, d_parent, d_count, status_word));
    return WAR_OK;
}

extern "C" war_status_t war_draft_pick(int32_t B, int32_t N, const int32_t* a_match_len, const int32_t* a_num_nodes,
                                       const int32_t* a_ids, const int32_t* a_parent, const int32_t* a_count,
                                       const int32_t* b_match_len, const int32_t* b_num_nodes, const int32_t* b_ids,
                                       const int32_t* b_parent, const int32_t* b_count, int32_t* d_source,
                                       int32_t* d_match_len, int32_t* d_num_nodes, int32_t* d_ids, int32_t* d_parent,
                                       int32_t* d_count, war_stream_t stream) {
    if (B < 0 || N < 1 || N > kMaxN) return WAR_ERR_INVALID_ARG;
    if (B == 0) return WAR_OK;
    if (!a_match_len || !a_num_nodes || !a_ids || !a_parent || !a_count || !b_match_len || !b_num_nodes || !b_ids || !b_parent ||
        !b_count || !d_source || !d_match_len || !d_num_nodes || !d_ids || !d_parent)
        return WAR_ERR_INVALID_ARG;
    war_draft_pick_kernel<<<(B + 7) / 8, 256, 0, stream>>>(B, N, a_match_len, a_num_nodes, a_ids, a_parent, a_count, b_match_len,
                                                          b_num_nodes, b_ids, b_parent, b_count, d_source, d_match_len,
                                                          d_num_nodes, d_ids, d_parent, d_count);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
