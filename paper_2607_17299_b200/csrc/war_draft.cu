// Draft: longest-suffix match against the suffix array, then best-first expansion of the matched
// interval into a frequency-ranked token tree.  One CTA per request.
//
// Match.  Lane l of warp 0 owns the candidate length l+1: it narrows the first-token bucket of its pattern
// to the suffix-array interval of the whole pattern with two binary searches.  The longest non-empty
// interval wins (occurrence is monotone in the length, so it is also the first empty one minus one).
//
// Tree.  A node is a suffix-array interval [lo, lo+cnt) whose suffixes share the first `depth` tokens.  Its
// children are the maximal runs between positions with lcp <= depth; a run's token is the suffix's token at
// `depth`, its count the run length.  Suffixes that end there (next entry is a separator) sort first, form
// runs of one, and are skipped.  Runs arrive in ascending token order, so keeping the first-seen run on equal
// counts is the (count descending, token ascending) rule.  Short intervals are scanned by warp 0, long ones
// by all warps over contiguous spans whose edge runs are stitched afterwards.  The pool of offered children
// lives in shared memory; the next slot is its maximum under (count desc, parent slot asc, token asc).
#include <climits>
#include "war_common.cuh"
#include "war_index.cuh"

namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxN = 64;
constexpr int kMaxK = 8;
constexpr int kMaxP = 32;
constexpr int kPoolCap = kMaxN * kMaxK;
constexpr int kBlockScanMin = 8192;          // intervals at least this long are scanned by every warp

struct TopK {                                 // warp-uniform, sorted by (cnt desc, start asc)
    int cnt[kMaxK];
    int start[kMaxK];
    int tok[kMaxK];
    int n;
};

__device__ __forceinline__ void topk_insert(TopK& t, int k, int cnt, int start, int tok) {
    // position = first entry that ranks below the newcomer
    int pos = t.n;
#pragma unroll
    for (int i = kMaxK - 1; i >= 0; --i)
        if (i < t.n && (cnt > t.cnt[i] || (cnt == t.cnt[i] && start < t.start[i]))) pos = i;
    if (pos >= k) return;
#pragma unroll
    for (int i = kMaxK - 1; i >= 1; --i)
        if (i > pos && i < k) { t.cnt[i] = t.cnt[i - 1]; t.start[i] = t.start[i - 1]; t.tok[i] = t.tok[i - 1]; }
#pragma unroll
    for (int i = 0; i < kMaxK; ++i)
        if (i == pos) { t.cnt[i] = cnt; t.start[i] = start; t.tok[i] = tok; }
    if (t.n < k) ++t.n;
}

// Bit t of the result: lcp byte t of the 16 loaded bytes is <= d.
__device__ __forceinline__ unsigned le_mask16(uint4 v, unsigned drep) {
    unsigned out = 0;
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const unsigned m = __vcmpleu4(w[i], drep);          // 0xff per byte that is <= d
        out |= ((m & 1u) | ((m >> 7) & 2u) | ((m >> 14) & 4u) | ((m >> 21) & 8u)) << (4 * i);
    }
    return out;
}

// One warp scans positions [sb, se) of the interval [lo, hi) at depth d.  Complete runs (both boundaries inside
// the span) go to the warp's top-k; the first and last boundary are returned for stitching.
__device__ void warp_scan_span(const uint8_t* __restrict__ lcp, const int32_t* __restrict__ sa,
                               const int32_t* __restrict__ corpus, int d, int sb, int se, int k, int lane,
                               TopK& tk, int& first_b, int& last_b) {
    tk.n = 0;
#pragma unroll
    for (int i = 0; i < kMaxK; ++i) { tk.cnt[i] = 0; tk.start[i] = 0; tk.tok[i] = 0; }
    int thr = 0;                                           // a run must beat this count to enter the top-k
    int carry = -1, my_first = -1;
    const unsigned drep = 0x01010101u * (unsigned)d;
    for (int base = sb & ~15; base < se; base += 512) {
        const int pos0 = base + lane * 16;
        unsigned bits = 0;
        if (pos0 < se) {
            const uint4 v = *reinterpret_cast<const uint4*>(lcp + pos0);
            bits = le_mask16(v, drep);
            if (pos0 < sb) bits &= ~((1u << (sb - pos0)) - 1u);
            if (pos0 + 16 > se) bits &= (1u << (se - pos0)) - 1u;
        }
        int last_pos = bits ? pos0 + 31 - __clz(bits) : -1;
        int incl = last_pos;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl = max(incl, y);
        }
        int prev = __shfl_up_sync(0xffffffffu, incl, 1);
        if (lane == 0) prev = -1;
        prev = max(prev, carry);
        carry = max(carry, __shfl_sync(0xffffffffu, incl, 31));
        // candidates in ascending position order: lowest lane first, ascending inside a lane
        bool have = false;
        int c_cnt = 0, c_start = 0;
        while (true) {
            if (!have) {
                while (bits) {
                    const int t = __ffs(bits) - 1;
                    bits &= bits - 1;
                    const int bpos = pos0 + t;
                    if (prev >= 0) {
                        const int c = bpos - prev;
                        if (c > thr) { c_cnt = c; c_start = prev; prev = bpos; have = true; break; }
                    } else {
                        my_first = bpos;
                    }
                    prev = bpos;
                }
            }
            const unsigned vote = __ballot_sync(0xffffffffu, have);
            if (!vote) break;
            const int src = __ffs(vote) - 1;
            const int cc = __shfl_sync(0xffffffffu, c_cnt, src);
            const int cs = __shfl_sync(0xffffffffu, c_start, src);
            if (lane == src) have = false;
            if (cc > thr) {
                const int tok = corpus[(int64_t)sa[cs] + d];
                if (tok >= 0) {
                    topk_insert(tk, k, cc, cs, tok);
#pragma unroll
                    for (int i = 0; i < kMaxK; ++i) if (i == k - 1 && tk.n == k) thr = tk.cnt[i];
                }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_first = max(my_first, __shfl_xor_sync(0xffffffffu, my_first, o));
    first_b = my_first;
    last_b = carry;
}

struct Shared {
    int pat[kMaxP];
    int pool_cnt[kPoolCap], pool_par[kPoolCap], pool_tok[kPoolCap], pool_lo[kPoolCap];
    int slot_lo[kMaxN], slot_cnt[kMaxN], slot_depth[kMaxN];
    int w_first[kWarps], w_last[kWarps], w_n[kWarps];
    int w_cnt[kWarps][kMaxK], w_start[kWarps][kMaxK], w_tok[kWarps][kMaxK];
    int fin_cnt[kMaxK], fin_start[kMaxK], fin_tok[kMaxK];
    int mode, cur, lo, cnt, depth, n_nodes, pool_n;
};

__device__ __forceinline__ int compare_suffix(const int32_t* __restrict__ corpus, int64_t s, const int* pat, int len) {
    // tokens 1 .. len-1 of the suffix at s against the pattern (token 0 is fixed by the bucket)
    for (int t = 1; t < len; ++t) {
        const int c = corpus[s + t];
        const int p = pat[t];
        if (c != p) return c < p ? -1 : 1;
    }
    return 0;
}

__global__ void __launch_bounds__(kThreads)
war_draft_kernel(const int32_t* __restrict__ corpus, const int32_t* __restrict__ sa, const uint8_t* __restrict__ lcp,
                 const int32_t* __restrict__ bucket, int vocab, const int32_t* __restrict__ tail,
                 const int32_t* __restrict__ tail_len, int P, int N, int K, int min_match,
                 int32_t* __restrict__ match_len, int32_t* __restrict__ num_nodes, int32_t* __restrict__ ids,
                 int32_t* __restrict__ parent, int32_t* __restrict__ count) {
    __shared__ Shared sh;
    const int b = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int32_t* o_ids = ids + (size_t)b * N;
    int32_t* o_par = parent + (size_t)b * N;
    int32_t* o_cnt = count ? count + (size_t)b * N : nullptr;

    if (tid < P) sh.pat[tid] = tail[(size_t)b * P + tid];
    __syncthreads();

    if (warp == 0) {
        // ---- longest-suffix match ----
        const int tl = min(max(tail_len[b], 0), P);
        const int len = lane + 1;
        int lo = 0, hi = 0;
        if (len <= tl) {
            const int* pat = sh.pat + (P - len);
            bool valid = true;
            for (int t = 0; t < len; ++t) valid = valid && pat[t] >= 0 && pat[t] < vocab;
            if (valid) {
                lo = bucket[pat[0]];
                hi = bucket[pat[0] + 1];
                if (len > 1 && hi > lo) {
                    int a = lo, z = hi;                          // lower bound: first suffix >= pattern
                    while (a < z) {
                        const int mid = a + ((z - a) >> 1);
                        if (compare_suffix(corpus, sa[mid], pat, len) < 0) a = mid + 1; else z = mid;
                    }
                    const int first = a;
                    z = hi;                                      // upper bound: first suffix > pattern
                    while (a < z) {
                        const int mid = a + ((z - a) >> 1);
                        if (compare_suffix(corpus, sa[mid], pat, len) <= 0) a = mid + 1; else z = mid;
                    }
                    lo = first;
                    hi = a;
                }
            }
        }
        const unsigned found = __ballot_sync(0xffffffffu, hi > lo);
        const int ml = found ? 32 - __clz(found) : 0;
        const int src = ml > 0 ? ml - 1 : 0;
        lo = __shfl_sync(0xffffffffu, lo, src);
        hi = __shfl_sync(0xffffffffu, hi, src);
        if (lane == 0) {
            const int c0 = ml > 0 ? hi - lo : 0;
            match_len[b] = ml;
            o_ids[0] = sh.pat[P - 1];
            o_par[0] = -1;
            if (o_cnt) o_cnt[0] = c0;
            sh.slot_lo[0] = lo; sh.slot_cnt[0] = c0; sh.slot_depth[0] = ml;
            sh.n_nodes = 1;
            sh.pool_n = 0;
            sh.cur = 0;
            const bool expand = ml >= max(1, min_match) && N > 1;
            sh.lo = lo; sh.cnt = c0; sh.depth = ml;
            sh.mode = !expand ? 0 : (c0 >= kBlockScanMin ? 2 : 1);
        }
    }

    // ---- best-first expansion ----
    while (true) {
        __syncthreads();
        const int mode = sh.mode;
        if (mode == 0) break;
        const int lo = sh.lo, cnt = sh.cnt, d = sh.depth, hi = lo + cnt;
        if (mode == 2) {
            const int a0 = lo & ~15;
            int span = (hi - a0 + kWarps - 1) / kWarps;
            span = (span + 511) & ~511;
            const int sb = max(lo, a0 + warp * span), se = min(hi, a0 + (warp + 1) * span);
            TopK tk;
            int fb = -1, lb = -1;
            tk.n = 0;
#pragma unroll
            for (int i = 0; i < kMaxK; ++i) { tk.cnt[i] = 0; tk.start[i] = 0; tk.tok[i] = 0; }
            if (sb < se) warp_scan_span(lcp, sa, corpus, d, sb, se, K, lane, tk, fb, lb);
            if (lane == 0) {
                sh.w_first[warp] = fb; sh.w_last[warp] = lb; sh.w_n[warp] = tk.n;
#pragma unroll
                for (int i = 0; i < kMaxK; ++i) { sh.w_cnt[warp][i] = tk.cnt[i]; sh.w_start[warp][i] = tk.start[i]; sh.w_tok[warp][i] = tk.tok[i]; }
            }
            __syncthreads();
        }
        if (warp == 0) {
            const int cur = sh.cur;
            int n_fin = 0;
            if (cnt == 1) {
                // a unique occurrence continues with the next corpus token, if the trajectory goes on
                if (lane == 0) {
                    const int tok = corpus[(int64_t)sa[lo] + d];
                    if (tok >= 0) { sh.fin_cnt[0] = 1; sh.fin_start[0] = lo; sh.fin_tok[0] = tok; n_fin = 1; }
                }
            } else {
                int nw = kWarps;
                if (mode == 1) {
                    TopK tk;
                    int fb, lb;
                    warp_scan_span(lcp, sa, corpus, d, lo, hi, K, lane, tk, fb, lb);
                    if (lane == 0) {
                        sh.w_first[0] = fb; sh.w_last[0] = lb; sh.w_n[0] = tk.n;
#pragma unroll
                        for (int i = 0; i < kMaxK; ++i) { sh.w_cnt[0][i] = tk.cnt[i]; sh.w_start[0][i] = tk.start[i]; sh.w_tok[0][i] = tk.tok[i]; }
                    }
                    nw = 1;
                }
                __syncwarp();
                if (lane == 0) {
                    // stitch the runs that cross span edges, then merge everything under (cnt desc, start asc)
                    auto offer = [&](int c, int s, int tok) {
                        int pos = n_fin;
                        for (int i = n_fin - 1; i >= 0; --i)
                            if (c > sh.fin_cnt[i] || (c == sh.fin_cnt[i] && s < sh.fin_start[i])) pos = i;
                        if (pos >= K) return;
                        if (tok == INT_MIN) { tok = corpus[(int64_t)sa[s] + d]; if (tok < 0) return; }
                        const int last = min(n_fin, K - 1);
                        for (int i = last; i > pos; --i) { sh.fin_cnt[i] = sh.fin_cnt[i - 1]; sh.fin_start[i] = sh.fin_start[i - 1]; sh.fin_tok[i] = sh.fin_tok[i - 1]; }
                        sh.fin_cnt[pos] = c; sh.fin_start[pos] = s; sh.fin_tok[pos] = tok;
                        if (n_fin < K) ++n_fin;
                    };
                    int carry = -1;
                    for (int w = 0; w < nw; ++w) {
                        if (sh.w_first[w] < 0) continue;
                        if (carry >= 0) offer(sh.w_first[w] - carry, carry, INT_MIN);
                        for (int e = 0; e < sh.w_n[w]; ++e) offer(sh.w_cnt[w][e], sh.w_start[w][e], sh.w_tok[w][e]);
                        carry = sh.w_last[w];
                    }
                    if (carry >= 0) offer(hi - carry, carry, INT_MIN);
                }
            }
            if (lane == 0) {
                int pn = sh.pool_n;
                for (int e = 0; e < n_fin && pn < kPoolCap; ++e, ++pn) {
                    sh.pool_cnt[pn] = sh.fin_cnt[e]; sh.pool_par[pn] = cur; sh.pool_tok[pn] = sh.fin_tok[e]; sh.pool_lo[pn] = sh.fin_start[e];
                }
                sh.pool_n = pn;
            }
            __syncwarp();
            // ---- take the best offer: count desc, parent slot asc, token asc ----
            const int pn = sh.pool_n;
            int bi = -1, bc = -1, bp = 0, bt = 0;
            for (int i = lane; i < pn; i += 32) {
                const int c = sh.pool_cnt[i], p = sh.pool_par[i], t = sh.pool_tok[i];
                if (bi < 0 || c > bc || (c == bc && (p < bp || (p == bp && t < bt)))) { bi = i; bc = c; bp = p; bt = t; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o), oc = __shfl_xor_sync(0xffffffffu, bc, o);
                const int op = __shfl_xor_sync(0xffffffffu, bp, o), ot = __shfl_xor_sync(0xffffffffu, bt, o);
                if (oi >= 0 && (bi < 0 || oc > bc || (oc == bc && (op < bp || (op == bp && ot < bt))))) { bi = oi; bc = oc; bp = op; bt = ot; }
            }
            if (lane == 0) {
                if (bi < 0) {
                    sh.mode = 0;
                } else {
                    const int j = sh.n_nodes;
                    const int slo = sh.pool_lo[bi];
                    const int last = pn - 1;
                    sh.pool_cnt[bi] = sh.pool_cnt[last]; sh.pool_par[bi] = sh.pool_par[last];
                    sh.pool_tok[bi] = sh.pool_tok[last]; sh.pool_lo[bi] = sh.pool_lo[last];
                    sh.pool_n = last;
                    o_ids[j] = bt; o_par[j] = bp;
                    if (o_cnt) o_cnt[j] = bc;
                    sh.slot_lo[j] = slo; sh.slot_cnt[j] = bc; sh.slot_depth[j] = sh.slot_depth[bp] + 1;
                    sh.n_nodes = j + 1;
                    if (j + 1 >= N) {
                        sh.mode = 0;
                    } else {
                        sh.cur = j; sh.lo = slo; sh.cnt = bc; sh.depth = sh.slot_depth[j];
                        sh.mode = bc >= kBlockScanMin ? 2 : 1;
                    }
                }
            }
        }
    }
    const int n = sh.n_nodes;
    if (tid == 0) num_nodes[b] = n;
    for (int j = n + tid; j < N; j += kThreads) {
        o_ids[j] = -1; o_par[j] = -1;
        if (o_cnt) o_cnt[j] = 0;
    }
}

}  // namespace

extern "C" war_status_t war_draft(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len,
                                  const war_draft_params_t* p, int32_t* d_match_len, int32_t* d_num_nodes,
                                  int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream) {
    if (!ix || !p) return WAR_ERR_INVALID_ARG;
    if (p->B < 0 || p->P < 1 || p->P > kMaxP || p->N < 1 || p->N > kMaxN || p->topk < 1 || p->topk > kMaxK || p->min_match < 0)
        return WAR_ERR_INVALID_ARG;
    if (p->P + p->N > ix->max_depth) return WAR_ERR_INVALID_ARG;     // the index is not ordered deep enough
    if (p->B == 0) return WAR_OK;
    if (!d_tail || !d_tail_len || !d_match_len || !d_num_nodes || !d_ids || !d_parent) return WAR_ERR_INVALID_ARG;
    war_draft_kernel<<<p->B, kThreads, 0, stream>>>(ix->corpus, ix->sa, ix->lcp, ix->bucket, ix->vocab, d_tail, d_tail_len,
                                                   p->P, p->N, p->topk, p->min_match, d_match_len, d_num_nodes, d_ids,
                                                   d_parent, d_count);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
