// Draft: longest-suffix match against the suffix array, then best-first expansion of the matched
// interval into a frequency-ranked token tree.  One CTA per request.
//
// Match.  Four lanes own each candidate length 1..32 (warps 0-3 the lower end of the pattern's suffix-array interval,
// warps 4-7 the upper end): a binary search inside the first token's bucket, pipelined two probes deep; lengths 2-5 are
// searched 33-way instead, by a warp each (warps 8-15).  The longest
// occurring length wins (occurrence is monotone in the length), and a length's search stops as soon as it is known not
// to matter (a shorter length does not occur, or a sufficiently longer one does).
//
// Tree.  A node is a suffix-array interval [lo, lo+cnt) whose suffixes share the first `depth` tokens.  Its
// children are the maximal runs between positions with lcp <= depth; a run's token is the suffix's token at
// `depth`, its count the run length.  Suffixes that end there (next entry is a separator) sort first, form
// runs of one, and are skipped.  Runs arrive in ascending token order, so keeping the first-seen run on equal
// counts is the (count descending, token ascending) rule.  Intervals of at most 32 suffixes are expanded in
// registers, longer ones are answered by the index's memo or scanned (by warp 0, the longest by all warps over
// contiguous spans whose edge runs are stitched afterwards).  The k offers of a slot form a sorted list in shared
// memory; the next slot is the best list head under (count desc, parent slot asc), which equals the rule
// (count desc, parent slot asc, token asc).  Warp 0 drives the expansion and meets the other warps at the block
// barrier only for the turns that need them.
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
constexpr int kMemoMinCount = 33;        // nodes with at least this many occurrences go through the index's memo
constexpr int kBlockScanMin = 1024;          // intervals at least this long are scanned by every warp (measured: 1024-2048 best)
constexpr int kLongRunFirstMin = 1024;       // intervals at least this long first look for runs of 16 or more only
constexpr int kWideFirst = 2, kWideLast = 5;  // candidate lengths searched 33-way by a warp of their own (warps 8-15)

struct TopK {                                 // warp-uniform, sorted by (cnt desc, start asc)
    int cnt[kMaxK];
    int start[kMaxK];
    int n;
};

__device__ __forceinline__ void topk_clear(TopK& t) {
    t.n = 0;
#pragma unroll
    for (int i = 0; i < kMaxK; ++i) { t.cnt[i] = 0; t.start[i] = 0; }
}

__device__ __forceinline__ void topk_insert(TopK& t, int k, int cnt, int start) {
    // position = first entry that ranks below the newcomer
    int pos = t.n;
#pragma unroll
    for (int i = kMaxK - 1; i >= 0; --i)
        if (i < t.n && (cnt > t.cnt[i] || (cnt == t.cnt[i] && start < t.start[i]))) pos = i;
    if (pos >= k) return;
#pragma unroll
    for (int i = kMaxK - 1; i >= 1; --i)
        if (i > pos && i < k) { t.cnt[i] = t.cnt[i - 1]; t.start[i] = t.start[i - 1]; }
#pragma unroll
    for (int i = 0; i < kMaxK; ++i)
        if (i == pos) { t.cnt[i] = cnt; t.start[i] = start; }
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

// One warp scans positions [sb, se) of a node's token range at depth d (suffixes that end at d are already cut
// off, so every run is a real continuation token).  Complete runs (both boundaries inside the span) go to the
// warp's top-k; the first and last boundary are returned for stitching.  No token is read here: a run is known by
// (count, start) and its token is looked up once, for the winners only.
//
// thr_shared is the largest "k-th best count" any warp of the CTA has published for this node: k runs at least
// that long exist somewhere in the node, so a run shorter than that cannot be among the node's k best (an equally
// long one still can, by its earlier start).  Once the bar is at 16 or more, no run that lies inside one lane's 16
// positions can pass it, and only the run ending at a lane's first boundary needs a look.
// (kept out of line, like the other rarely taken paths below: the kernel's hot path is one warp walking a long chain of
// dependent steps, and it runs at the speed of the instruction cache unless the code it crosses stays small)
__device__ __noinline__ void warp_scan_span(const uint8_t* __restrict__ lcp, int d, int sb, int se, int k, int lane,
                               TopK& tk, int& first_b, int& last_b, int* thr_shared) {
    topk_clear(tk);
    int thr_local = 0;                                     // a run must beat this count to enter this warp's top-k
    int carry = -1, my_first = -1;
    const unsigned drep = 0x01010101u * (unsigned)d;
    constexpr int kAhead = 4;                               // 16-byte loads in flight per lane (2 KB per warp step)
    for (int base0 = sb & ~15; base0 < se; base0 += 512 * kAhead) {
        uint4 v[kAhead];
#pragma unroll
        for (int q = 0; q < kAhead; ++q) {
            const int p0 = base0 + q * 512 + lane * 16;
            v[q] = p0 < se ? *reinterpret_cast<const uint4*>(lcp + p0) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int q = 0; q < kAhead; ++q) {
            const int base = base0 + q * 512;
            if (base >= se) break;                              // warp-uniform
            const int pos0 = base + lane * 16;
            unsigned bits = 0;
            if (pos0 < se) {
                bits = le_mask16(v[q], drep);
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
            int thr = max(thr_local, *(volatile int*)thr_shared - 1);
            thr = __shfl_sync(0xffffffffu, thr, 0);                // one value for the whole warp
            if (bits && prev < 0) my_first = pos0 + __ffs(bits) - 1;  // the span's very first boundary opens, closes nothing
            if (thr >= 15) {
                // only the run that ends at a lane's first boundary can be long enough: one proposal per lane
                int c = 0, st = 0;
                if (bits && prev >= 0) { c = pos0 + __ffs(bits) - 1 - prev; st = prev; }
                while (true) {
                    // best proposal of the warp under (count desc, start asc)
                    int bc = c > thr ? c : 0, bs = st;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const int oc = __shfl_xor_sync(0xffffffffu, bc, o), os = __shfl_xor_sync(0xffffffffu, bs, o);
                        if (oc > bc || (oc == bc && oc > 0 && os < bs)) { bc = oc; bs = os; }
                    }
                    if (bc == 0) break;
                    topk_insert(tk, k, bc, bs);
                    if (c == bc && st == bs) c = 0;
                    if (tk.n == k) {
#pragma unroll
                        for (int i = 0; i < kMaxK; ++i) if (i == k - 1) thr_local = tk.cnt[i];
                        if (lane == 0) atomicMax(thr_shared, thr_local);
                        thr = max(thr, thr_local);
                    }
                }
            } else {
                // Dense case.  Every lane walks its own boundaries (all lanes at once) and proposes its best run that
                // still beats the bar; the warp takes the best proposal, raises the bar, and asks again.  At most k
                // rounds per chunk can succeed, so the cost stays bounded however many tiny runs there are.
                // len[t]: length of the run that ends at this lane's position t (0: no boundary there, or nothing opened it)
                int len[16];
                {
                    int p = prev;
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const bool bd = (bits >> t) & 1u;
                        len[t] = (bd && p >= 0) ? pos0 + t - p : 0;
                        p = bd ? pos0 + t : p;
                    }
                }
                while (true) {
                    int c = 0, ct = 0;
#pragma unroll
                    for (int t = 0; t < 16; ++t)
                        if (len[t] > thr && len[t] > c) { c = len[t]; ct = t; }      // strict: the earliest of equal runs
                    const int st = pos0 + ct - c;
                    int bc = c, bs = st;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const int oc = __shfl_xor_sync(0xffffffffu, bc, o), os = __shfl_xor_sync(0xffffffffu, bs, o);
                        if (oc > bc || (oc == bc && oc > 0 && os < bs)) { bc = oc; bs = os; }
                    }
                    if (bc == 0) break;
                    topk_insert(tk, k, bc, bs);
                    if (c == bc && st == bs) {
#pragma unroll
                        for (int t = 0; t < 16; ++t) if (t == ct) len[t] = 0;            // taken
                    }
                    if (tk.n == k) {
#pragma unroll
                        for (int i = 0; i < kMaxK; ++i) if (i == k - 1) thr_local = tk.cnt[i];
                        if (lane == 0) atomicMax(thr_shared, thr_local);
                        thr = max(thr, thr_local);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_first = max(my_first, __shfl_xor_sync(0xffffffffu, my_first, o));
    first_b = my_first;
    last_b = carry;
}

// Number of suffixes of the interval [lo, hi) whose entry at depth d is a separator (the occurrence ends its
// trajectory there).  They sort before every real token, so this is the first position holding a token >= 0,
// found by a 32-way search of one warp; almost always the very first probe answers.
__device__ __noinline__ int count_ending(const int32_t* __restrict__ corpus, const int32_t* __restrict__ sa, int lo, int hi, int d, int lane) {
    int first = corpus[(int64_t)sa[lo] + d];
    if (first >= 0) return 0;
    int a = lo + 1, z = hi;                                 // answer in [a, z]: positions < a hold separators
    while (a < z) {
        const int span = z - a;
        const int step = (span + 31) / 32;
        const int pos = min(a + lane * step, z - 1);
        const bool sep = corpus[(int64_t)sa[pos] + d] < 0;
        const unsigned m = __ballot_sync(0xffffffffu, !sep);
        if (m == 0) { a = min(a + 31 * step, z - 1) + 1; continue; }
        const int f = __ffs(m) - 1;                          // first probe holding a real token
        z = min(a + f * step, z - 1);
        a = f == 0 ? a : min(a + (f - 1) * step, z - 1) + 1;
        if (f == 0) break;
    }
    return z - lo;
}

struct Shared {
    int pat[kMaxP];
    // offers: the rank-r continuation of slot j sits at j * kMaxK + r, a slot's offers in the order (count desc, token asc);
    // count 0 ends a slot's list
    int pool_cnt[kPoolCap], pool_tok[kPoolCap], pool_lo[kPoolCap];
    int slot_depth[kMaxN];
    int w_first[kWarps], w_last[kWarps], w_n[kWarps];
    int w_cnt[kWarps][kMaxK], w_start[kWarps][kMaxK];
    int st_cnt[32], st_start[32];               // runs that cross span edges (one per span) and the closing run
    int fin_cnt[kMaxK], fin_start[kMaxK], fin_tok[kMaxK];
    int mode, cur, lo, cnt, depth, n_nodes, thr_shared, long_runs_only, full_lo, full_cnt;
    int n_running, n_cap;
    int m_lo[32], m_hi[32], m_occ[32];          // per candidate length: interval [lo, hi) of its pattern, occurs
    int min_fail, max_ok;                       // smallest length known not to occur, largest length known to occur
    int memo_slot;                              // >= 0: the node being expanded goes into this memo entry when it is done
    // a batch of small nodes created in one round (equal counts), expanded by one warp each
    int it_slot[kWarps], it_lo[kWarps], it_cnt[kWarps], it_depth[kWarps], n_items;
};

// kCtasPerSm = 2: 64 registers per thread, 296 requests in one wave; 1: 128 registers (nothing spills), used when the
// grid fits the SMs anyway, which is the low-load case where this kernel's latency matters most.
template <int kCtasPerSm>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
war_draft_kernel(const int32_t* __restrict__ corpus, const war_index_view* __restrict__ view, int vocab, const int32_t* __restrict__ tail,
                 const int32_t* __restrict__ tail_len, int B, int P, int N, int K, int min_match, int spec_batch_limit,
                 int fac_num, int fac_den, int prob_num, int prob_den, int32_t* __restrict__ match_len, int32_t* __restrict__ num_nodes, int32_t* __restrict__ ids,
                 int32_t* __restrict__ parent, int32_t* __restrict__ count, int32_t* __restrict__ cand_len) {
    __shared__ Shared sh;
    const int b = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The index arrays come from the set that is published NOW (not when the launch was enqueued or captured): the
    // request for them goes out first and is in flight while the tail is read.
    const war_index_arrays arrays = view->set[*(const volatile unsigned int*)&view->cur & 1u];
    const int32_t* __restrict__ sa = arrays.sa;
    const uint8_t* __restrict__ lcp = arrays.lcp;
    const int32_t* __restrict__ bucket = arrays.bucket;
    int32_t* memo = arrays.memo;
    // Scoring several suffix lengths: CTA (b, c) drafts request b from the suffix that is c tokens shorter than the
    // longest match and leaves its tree in row b * gridDim.y + c of the candidate arrays (all output pointers then
    // address those); a second kernel picks the winner.  With one candidate per request the row is the request.
    const int cand = blockIdx.y;
    const size_t row = (size_t)b * gridDim.y + cand;
    int32_t* o_ids = ids + row * N;
    int32_t* o_par = parent + row * N;
    int32_t* o_cnt = count ? count + row * N : nullptr;

    if (tid < P) sh.pat[tid] = tail[(size_t)b * P + tid];
    if (tid == 0) { sh.min_fail = kMaxP + 1; sh.max_ok = 0; }
    // Workload-aware switch: a request with tail_len < 0 is not running; when more requests run than the limit,
    // nothing is looked up and every running request gets the root alone (a plain decode step through the same
    // calls).  Every CTA counts the running requests itself: no extra launch, no state between calls.
    bool plain = false;
    if (spec_batch_limit > 0) {
        int c = 0;
        for (int i = tid; i < B; i += kThreads) c += tail_len[i] >= 0;
        if (tid == 0) sh.n_running = 0;
        __syncthreads();
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if (lane == 0 && c) atomicAdd(&sh.n_running, c);
        __syncthreads();
        plain = sh.n_running > spec_batch_limit;
    }
    __syncthreads();
    const int my_tl = tail_len[b];
    if (my_tl < 0 || plain) {
        const int n = my_tl < 0 ? 0 : 1;
        if (tid == 0) {
            match_len[row] = 0; num_nodes[row] = n;
            if (cand_len) cand_len[row] = cand == 0 ? 0 : -1;            // one candidate: the root alone (or nothing)
            if (n) { o_ids[0] = sh.pat[P - 1]; o_par[0] = -1; if (o_cnt) o_cnt[0] = 0; }
        }
        for (int j = n + tid; j < N; j += kThreads) {
            o_ids[j] = -1; o_par[j] = -1;
            if (o_cnt) o_cnt[j] = 0;
        }
        return;
    }

    // The node warp 0 works on next, in its registers (uniform across the lanes): slot, token range (the interval minus
    // the suffixes that end at this depth), depth, whole interval, memo entry to fill (-1 none), kind of turn, and for
    // a memo hit the number of offers and the occurrences they cover.  What other warps read is mirrored in shared memory.
    int t_cur = 0, t_lo = 0, t_cnt = 0, t_depth = 0, t_full_lo = 0, t_full_cnt = 0, t_memo_slot = -1, t_mode = 0, t_nfin = 0, t_cov = 0;
    auto publish = [&](int slot, int lo, int cnt, int depth) {          // warp 0, all lanes
        t_cur = slot; t_lo = lo; t_cnt = cnt; t_depth = depth; t_full_lo = lo; t_full_cnt = cnt; t_memo_slot = -1;
        if (cnt <= 32) {                                                // handled in registers, one suffix per lane
            t_mode = 3;
            if (lane == 0) sh.mode = 3;
            return;
        }
        // Large nodes are looked up in the index's memo first (same node, same k => same answer for every request)
        if (cnt >= kMemoMinCount) {
            const unsigned long long key = ((unsigned long long)(unsigned)(lo + 1) << 16) | ((unsigned long long)depth << 8) | (unsigned)K;
            unsigned h = (unsigned)(key * 0x9E3779B97F4A7C15ull >> 40) & (kMemoEntries - 1);
            // One coalesced read of the whole 128-byte entry (plus the key as one 64-bit word on lane 0).  Payload
            // words are stored with 1 added and the table starts zeroed, so every word says by itself whether it has
            // been written: a hit needs the key and all words it uses to be there, in whatever order they arrived.
            volatile int32_t* en = memo + (size_t)h * kMemoInts;
            unsigned long long got = 0ull;
            if (lane == 0) got = *(volatile unsigned long long*)en;
            const int word = en[lane];
            got = __shfl_sync(0xffffffffu, got, 0);
            if (got == key) {
                const int n_fin = __shfl_sync(0xffffffffu, word, 3) - 1;
                const int r = (lane - 4) & 7;                            // lanes 4..11 counts, 12..19 starts, 20..27 tokens
                const bool mine = lane >= 4 && lane < 28 && r < n_fin;  // a word this node's answer uses
                if (n_fin >= 0 && __ballot_sync(0xffffffffu, mine && word == 0) == 0u) {
                    // the answer goes straight into this slot's offer list
                    const int at = slot * kMaxK + r;
                    if (lane >= 4 && lane < 12) {
                        const bool keep = mine && (prob_num == 0 || (long long)word * prob_den >= (long long)prob_num * cnt);
                        sh.pool_cnt[at] = keep ? word : 0;
                    } else if (mine) {
                        if (lane < 20) sh.pool_lo[at] = word - 1; else sh.pool_tok[at] = word - 1;
                    }
                    __syncwarp();
                    t_nfin = n_fin;
                    t_cov = __reduce_add_sync(0xffffffffu, mine && lane < 12 ? word : 0);
                    t_mode = 4;
                    if (lane == 0) sh.mode = 4;
                    return;
                }
            } else if (got == 0ull) {
                t_memo_slot = (int)h;                                    // free: this expansion will try to fill it
            }
        }
        const int e = count_ending(corpus, sa, lo, lo + cnt, depth, lane);
        t_lo = lo + e; t_cnt = cnt - e;
        // Large nodes are first scanned for runs of 16 positions or more only (bar preset to 16): that pass never
        // walks the boundaries inside a lane.  It is exact whenever it finds k such runs; otherwise the node is
        // scanned again without the preset.
        const int long_first = (cnt - e) >= kLongRunFirstMin;
        t_mode = (cnt - e) >= kBlockScanMin ? 2 : 1;
        if (lane == 0) {
            sh.lo = lo + e; sh.cnt = cnt - e; sh.depth = depth;
            sh.long_runs_only = long_first;
            sh.thr_shared = long_first ? 16 : 0;
            sh.mode = t_mode;
        }
    };

    // Warp 0's running state of the expansion lives in registers (uniform across its lanes unless noted), so that taking
    // the next offer waits for no shared-memory round trip: slots made so far, slot budget, and per lane the offer lists
    // of slots lane and lane + 32: how many of a list's offers were taken (cur) and the count of its next one (head, 0 =
    // none left).  A list is sorted, so the best offer of all is the best head: count desc, then the smaller slot.
    int n_nodes = 1, n_cap = N, head0 = 0, head1 = 0, cur0 = 0, cur1 = 0;
    // Rank of a run among the runs of a small node under (length desc, lane asc): c = run length on head lanes (<= 32),
    // 0 elsewhere.  Six ballots, one per bit of the length, instead of one warp arg-max per winner.
    auto run_rank = [&](int c) -> int {
        unsigned gt = 0, eq = 0xffffffffu;
#pragma unroll
        for (int bit = 5; bit >= 0; --bit) {
            const unsigned m = __ballot_sync(0xffffffffu, (c >> bit) & 1);
            if ((c >> bit) & 1) eq &= m; else { gt |= eq & m; eq &= ~m; }
        }
        return __popc(gt) + __popc(eq & ((1u << lane) - 1u));
    };

    // ---- longest-suffix match ----
    // Warps 0-3 find the lower end of every candidate length's interval, warps 4-7 at the same time the upper end: four
    // lanes per length (thread t: length (t % 128) / 4 + 1, every fourth token from t % 4 on behind the known common
    // prefix), so one probe of a binary search compares up to 32 tokens in a single memory latency whatever the depth of
    // the match.  The four lanes of a group hold the same search state.
    // Occurrence is monotone in the length, and only the longest occurring length (and, when several lengths are
    // scored, the few below it) is drafted from.  So a search is given up as soon as it cannot matter: every group
    // posts its verdict the moment it has one (largest length seen to occur, smallest seen not to), and a group whose
    // length lies above the latter or too far below the former stops probing.  The searches take as many steps as
    // their buckets are deep (up to 22 on a frequent token against 10 on an average one), one memory latency each,
    // so this ends the phase with the deepest bucket among the lengths that count instead of among all 32.
    const int tl = min(max(my_tl, 0), P);
    if (warp < 8) {
        const bool upper = warp >= 4;                             // first suffix above every suffix that starts with the pattern
        const int len = ((tid & 127) >> 2) + 1, part = tid & 3;
        const int* pat = sh.pat + (P - len);
        int lo = 0, bucket_hi = 0;
        bool occurs = false, searching = false;
        const bool wide = len >= kWideFirst && len <= kWideLast && len <= tl;    // a warp of its own searches this length
        if (len <= tl && !wide) {
            bool valid = true;
            for (int t = 0; t < len; ++t) valid = valid && pat[t] >= 0 && pat[t] < vocab;
            if (valid) {
                lo = bucket[pat[0]];
                bucket_hi = bucket[pat[0] + 1];
                occurs = bucket_hi > lo;
                searching = len > 1 && occurs;
            }
        }
        const int keep_below = (int)gridDim.y - 1;                // lengths this far below the longest match are still drafted from
        if (!upper && part == 0 && !searching && !wide) {         // decided without a search
            if (occurs) atomicMax(&sh.max_ok, len); else atomicMin(&sh.min_fail, len);
        }
        bool given_up = false;
        // bound by binary search; it remembers how many tokens the pattern shares with the suffixes at its
        // current ends, so comparisons restart there (all bucket members share token 0).  The search is pipelined two
        // probes deep so that a step costs one memory latency instead of two or three: while the current probe is
        // compared, the first tokens of BOTH possible next probes are on their way (their suffix-array entries came
        // in during the previous step), and so are the suffix-array entries of the four probes after those.  The loop
        // runs while any group of the warp still searches (full-warp shuffles).
        int a = searching ? lo : 0, z = searching ? bucket_hi : 0, ma = 1, mz = 1;
        int mid = a + ((z - a) >> 1);
        int s_mid = 0, s_l = 0, s_r = 0, c0 = 0, c1 = 0, at = 1 + part;   // at: pattern position of c0 (c1 is 4 further)
        if (searching) {
            const int mid_l = a + ((mid - a) >> 1), mid_r = mid + 1 + ((z - mid - 1) >> 1);
            s_mid = sa[mid];                                      // the bucket is not empty
            s_l = a < mid ? sa[mid_l] : 0;
            s_r = mid + 1 < z ? sa[mid_r] : 0;
            c0 = at < len ? corpus[(int64_t)s_mid + at] : 0;
            c1 = at + 4 < len ? corpus[(int64_t)s_mid + at + 4] : 0;
        }
        int seen_fail = kMaxP + 1, seen_ok = 0;                   // the two verdict words as read during the previous step
        while (__any_sync(0xffffffffu, a < z)) {                  // first suffix >= pattern (upper: > every match)
            if (a < z && (len > seen_fail || len < seen_ok - keep_below)) {
                z = a;                                            // this length no longer matters
                given_up = true;
            }
            const bool active = a < z;
            const int mid_l = a + ((mid - a) >> 1), mid_r = mid + 1 + ((z - mid - 1) >> 1);
            const bool has_l = active && a < mid, has_r = active && mid + 1 < z;
            // suffix-array entries two steps ahead
            const int mid_ll = a + ((mid_l - a) >> 1), mid_lr = mid_l + 1 + ((mid - mid_l - 1) >> 1);
            const int mid_rl = mid + 1 + ((mid_r - mid - 1) >> 1), mid_rr = mid_r + 1 + ((z - mid_r - 1) >> 1);
            const int s_ll = has_l && a < mid_l ? sa[mid_ll] : 0, s_lr = has_l && mid_l + 1 < mid ? sa[mid_lr] : 0;
            const int s_rl = has_r && mid + 1 < mid_r ? sa[mid_rl] : 0, s_rr = has_r && mid_r + 1 < z ? sa[mid_rr] : 0;
            // first tokens of both possible next probes, from the prefix known now (it can only grow)
            const int from = min(ma, mz), nt = from + part;
            const int l0 = has_l && nt < len ? corpus[(int64_t)s_l + nt] : 0, l1 = has_l && nt + 4 < len ? corpus[(int64_t)s_l + nt + 4] : 0;
            const int r0 = has_r && nt < len ? corpus[(int64_t)s_r + nt] : 0, r1 = has_r && nt + 4 < len ? corpus[(int64_t)s_r + nt + 4] : 0;
            // the verdicts so far ride along with this step's loads and are looked at when the next step begins, where
            // the step waits for those loads anyway (a wait of their own anywhere else costs the step a second latency)
            seen_fail = *(volatile int*)&sh.min_fail;
            seen_ok = *(volatile int*)&sh.max_ok;
            // first differing position of the group (position * 2 + "corpus token smaller"); 2 * len = none differs.
            // Eight tokens first: most probes differ there; the rest (up to 24 more) only for the groups that need them.
            int key;
            {
                const int q0 = pat[min(at, len - 1)], q1 = pat[min(at + 4, len - 1)];
                const bool d0 = at < len && c0 != q0, d1 = at + 4 < len && c1 != q1;
                key = d0 ? (at << 1) | (int)(c0 < q0) : d1 ? ((at + 4) << 1) | (int)(c1 < q1) : (len << 1);
                key = min(key, __shfl_xor_sync(0xffffffffu, key, 1));
                key = min(key, __shfl_xor_sync(0xffffffffu, key, 2));
            }
            const int t0 = at + 8;                                                // the group's tokens so far: [at - part, + 8)
            const bool more = active && key == (len << 1) && t0 - part < len;    // the same for the lanes of a group
            if (__any_sync(0xffffffffu, more)) {
                unsigned ne = 0, lt = 0;
                int c[6];
#pragma unroll
                for (int i = 0; i < 6; ++i) c[i] = (more && t0 + 4 * i < len) ? corpus[(int64_t)s_mid + t0 + 4 * i] : 0;
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const int q = pat[min(t0 + 4 * i, len - 1)];
                    ne |= (unsigned)(t0 + 4 * i < len && c[i] != q) << i;
                    lt |= (unsigned)(c[i] < q) << i;
                }
                const int f = __ffs(ne) - 1;
                int key2 = ne ? ((t0 + 4 * f) << 1) | (int)((lt >> f) & 1u) : (len << 1);
                key2 = min(key2, __shfl_xor_sync(0xffffffffu, key2, 1));
                key2 = min(key2, __shfl_xor_sync(0xffffffffu, key2, 2));
                if (more) key = key2;
            }
            if (active) {
                const int m = key >> 1;                             // leading tokens that agree
                if (m < len ? (key & 1) != 0 : upper) { a = mid + 1; ma = m; mid = mid_r; s_mid = s_r; c0 = r0; c1 = r1; s_l = s_rl; s_r = s_rr; }
                else { z = mid; mz = m; mid = mid_l; s_mid = s_l; c0 = l0; c1 = l1; s_l = s_ll; s_r = s_lr; }
                at = nt;
                if (a >= z && !upper && part == 0) {               // this search has just ended: post its verdict
                    if (a < bucket_hi && mz == len) atomicMax(&sh.max_ok, len); else atomicMin(&sh.min_fail, len);
                }
            }
        }
        if (!upper) {
            if (searching) {
                lo = a;
                // the pattern occurs iff the suffix there starts with it: that suffix was the last probe that was not
                // below the pattern, and mz tokens of it agreed (a search that was given up reports nothing: its
                // length is either above the longest match or below every length that is drafted from)
                occurs = !given_up && lo < bucket_hi && mz == len;
            }
            if (part == 0 && !wide) { sh.m_lo[len - 1] = lo; sh.m_occ[len - 1] = occurs; }
        } else if (part == 0 && !wide) {
            sh.m_hi[len - 1] = searching ? a : bucket_hi;         // a one-token pattern's interval is its bucket
        }
    } else {
        // Warps 8-15: the short candidate lengths, the ones that nearly always decide the match (the typical longest
        // match is two to four tokens, and the search of the first length that fails is what releases all longer
        // ones).  A warp per length and interval end narrows the bucket 33-way: every lane probes one suffix (its
        // suffix-array entry, then the pattern's few tokens, all in flight together: two memory latencies per step)
        // and the ballot of "sorts below the end that is looked for" picks the sub-interval.  A bucket of 2^21
        // suffixes takes 5 steps = 10 latencies instead of the binary search's 21.
        const int len = kWideFirst + ((warp - 8) & 3);
        const bool upper = warp >= 12;
        if (len <= tl) {
            const int* pat = sh.pat + (P - len);
            bool valid = true;
            for (int t = 0; t < len; ++t) valid = valid && pat[t] >= 0 && pat[t] < vocab;
            int a = 0, z = 0, bucket_hi = 0;
            if (valid) { a = bucket[pat[0]]; bucket_hi = z = bucket[pat[0] + 1]; }
            bool z_starts = false, given_up = false;              // z_starts: the suffix at z starts with the pattern
            int q[kWideLast];
            for (int t = 1; t < kWideLast; ++t) q[t] = t < len ? pat[t] : 0;
            while (a < z) {
                if (len > *(volatile int*)&sh.min_fail) { given_up = true; break; }
                const int n = z - a;
                const bool last = n <= 32;
                const int pos = last ? a + lane : a + (int)(((unsigned long long)(lane + 1) * (unsigned)n) / 33u);
                const bool live = !last || lane < n;
                int cmp = 0;                                      // -1 the suffix sorts below the pattern, 0 starts with it, 1 above
                if (live) {
                    const int64_t sfx = sa[pos];
                    int c[kWideLast];
#pragma unroll
                    for (int t = 1; t < kWideLast; ++t) c[t] = t < len ? corpus[sfx + t] : 0;
#pragma unroll
                    for (int t = 1; t < kWideLast; ++t)
                        if (t < len && cmp == 0 && c[t] != q[t]) cmp = c[t] < q[t] ? -1 : 1;
                }
                const unsigned below = __ballot_sync(0xffffffffu, live && (upper ? cmp <= 0 : cmp < 0));
                const unsigned starts = __ballot_sync(0xffffffffu, live && cmp == 0);
                const int cnt = __popc(below);                    // the suffixes are sorted: the lanes below form a prefix
                const int pos_prev = __shfl_sync(0xffffffffu, pos, max(cnt - 1, 0));
                const int pos_next = __shfl_sync(0xffffffffu, pos, min(cnt, 31));
                if (last) {
                    if (cnt < n) z_starts = (starts >> cnt) & 1u;
                    a = z = a + cnt;
                } else {
                    if (cnt < 32) { z = pos_next; z_starts = (starts >> cnt) & 1u; }
                    if (cnt > 0) a = pos_prev + 1;
                }
            }
            if (lane == 0) {
                if (!upper) {
                    const bool occurs = valid && !given_up && a < bucket_hi && z_starts;
                    sh.m_lo[len - 1] = a; sh.m_occ[len - 1] = occurs;
                    if (!given_up) { if (occurs) atomicMax(&sh.max_ok, len); else atomicMin(&sh.min_fail, len); }
                } else {
                    sh.m_hi[len - 1] = a;
                }
            }
        }
    }
    __syncthreads();
    if (warp == 0) {
        int lo = sh.m_lo[lane], hi = sh.m_hi[lane];
        const bool occurs = sh.m_occ[lane] != 0;
        const unsigned found = __ballot_sync(0xffffffffu, occurs);
        const int ml_longest = found ? 32 - __clz(found) : 0;
        // candidate c drafts from the suffix of ml_longest - c tokens (every shorter suffix of an occurring string
        // occurs, and its lane holds that suffix's interval); lengths below max(1, min_match) are no candidates
        const int ml = ml_longest - cand;
        if (cand > 0 && ml < max(1, min_match)) {
            n_nodes = 0;
            if (lane == 0) { match_len[row] = ml_longest; cand_len[row] = -1; sh.n_nodes = 0; sh.mode = 0; }
        } else {
        const int src = ml > 0 ? ml - 1 : 0;
        lo = __shfl_sync(0xffffffffu, lo, src);
        hi = __shfl_sync(0xffffffffu, hi, src);
        const int c0 = ml > 0 ? hi - lo : 0;
        // node budget: a longer match earns a larger tree (at most 1 + floor(match_len * fac_num / fac_den) slots)
        n_cap = fac_num > 0 ? min(N, 1 + (int)(((long long)ml * fac_num) / fac_den)) : N;
        const bool expand = ml >= max(1, min_match) && n_cap > 1;
        if (lane == 0) {
            sh.n_cap = n_cap;
            match_len[row] = ml_longest;
            if (cand_len) cand_len[row] = ml;
            o_ids[0] = sh.pat[P - 1];
            o_par[0] = -1;
            if (o_cnt) o_cnt[0] = c0;
            sh.slot_depth[0] = ml;
            sh.n_nodes = 1;
            sh.mode = 0;
        }
        if (expand) publish(0, lo, c0, ml);
        }
    }

    // ---- best-first expansion ----
    // Modes: 1 a node scanned by warp 0 alone, 2 a node scanned by all warps, 3 a node of at most 32 suffixes (in
    // registers), 4 a node answered by the memo, 6 a batch of small nodes (one per warp).  Only 2 and 6 need the other
    // warps: they wait at the barrier below while warp 0 works through nodes of the other kinds on its own.
    while (true) {
        __syncthreads();
        int mode = sh.mode;
        if (mode == 0) break;
        if (mode == 6) {
            // A batch of small nodes: warp w expands item w in registers (one suffix per lane) and adds its k best
            // continuations to the offer pool.
            if (warp < sh.n_items) {
                const int j = sh.it_slot[warp], ilo = sh.it_lo[warp], icnt = sh.it_cnt[warp], idp = sh.it_depth[warp];
                const int tok = lane < icnt ? corpus[(int64_t)sa[ilo + lane] + idp] : -1;
                const int prev_tok = __shfl_up_sync(0xffffffffu, tok, 1);
                const bool real = lane < icnt && tok >= 0;
                const bool head = real && (lane == 0 || tok != prev_tok);
                const unsigned hm = __ballot_sync(0xffffffffu, head);
                const unsigned vm = __ballot_sync(0xffffffffu, real);
                const int end = vm ? 32 - __clz(vm) : 0;
                const unsigned after = (hm >> 1) >> lane;
                int c = head ? (after ? lane + __ffs(after) : end) - lane : 0;
                const int rank = run_rank(c);
                if (head && rank < K) {
                    const bool keep = prob_num == 0 || (long long)c * prob_den >= (long long)prob_num * icnt;
                    const int at = j * kMaxK + rank;
                    sh.pool_cnt[at] = keep ? c : 0; sh.pool_tok[at] = tok; sh.pool_lo[at] = ilo + lane;
                }
                const int n_runs = min(K, __popc(hm));
                if (lane >= n_runs && lane < kMaxK) sh.pool_cnt[j * kMaxK + lane] = 0;
            }
            __syncthreads();
        }
        if (mode == 2) {
            const int lo = sh.lo, d = sh.depth, hi = lo + sh.cnt;
            const int a0 = lo & ~15;
            int span = (hi - a0 + kWarps - 1) / kWarps;
            span = (span + 511) & ~511;
            const int sb = max(lo, a0 + warp * span), se = min(hi, a0 + (warp + 1) * span);
            TopK tk;
            int fb = -1, lb = -1;
            topk_clear(tk);
            if (sb < se) warp_scan_span(lcp, d, sb, se, K, lane, tk, fb, lb, &sh.thr_shared);
            if (lane == 0) {
                sh.w_first[warp] = fb; sh.w_last[warp] = lb; sh.w_n[warp] = tk.n;
#pragma unroll
                for (int i = 0; i < kMaxK; ++i) { sh.w_cnt[warp][i] = tk.cnt[i]; sh.w_start[warp][i] = tk.start[i]; }
            }
            __syncthreads();
        }
        if (warp == 0) {
            while (true) {                                               // one node (or batch) per turn
            __syncwarp();                                                // single-lane stores end here: the lanes go on together
            const int lo = t_lo, cnt = t_cnt, d = t_depth, hi = lo + cnt, cur = t_cur;
            if (mode == 6) {
                // the batch's warps wrote the lists of slots it_slot[0 .. n_items): their owners pick up the heads
                const int j_first = sh.it_slot[0];
                const int jj = j_first + ((lane - j_first) & 31);
                if (jj < j_first + sh.n_items) {
                    const int h = sh.pool_cnt[jj * kMaxK];
                    if (jj < 32) { head0 = h; cur0 = 0; } else { head1 = h; cur1 = 0; }
                }
            } else {
            int n_fin = 0, covered = 0;
            if (mode == 3) {
                // at most 32 suffixes: lane i reads the continuation token of suffix lo+i; suffixes that end here hold a
                // separator (negative) and sort first; equal tokens are adjacent, so a run is a head lane plus followers
                const int tok = lane < cnt ? corpus[(int64_t)sa[lo + lane] + d] : -1;
                const int prev_tok = __shfl_up_sync(0xffffffffu, tok, 1);
                const bool real = lane < cnt && tok >= 0;
                const bool head = real && (lane == 0 || tok != prev_tok);
                const unsigned hm = __ballot_sync(0xffffffffu, head);
                const unsigned vm = __ballot_sync(0xffffffffu, real);
                const int end = vm ? 32 - __clz(vm) : 0;
                const unsigned after = (hm >> 1) >> lane;                  // heads strictly after this lane
                int c = head ? (after ? lane + __ffs(after) : end) - lane : 0;
                const int rank = run_rank(c);
                const bool win = head && rank < K;                        // the k longest runs, each written by its head lane
                if (win) {
                    const bool keep = prob_num == 0 || (long long)c * prob_den >= (long long)prob_num * cnt;
                    const int at = cur * kMaxK + rank;
                    sh.pool_cnt[at] = keep ? c : 0; sh.pool_tok[at] = tok; sh.pool_lo[at] = lo + lane;
                }
                n_fin = min(K, __popc(hm));
                covered = __reduce_add_sync(0xffffffffu, win ? c : 0);
                if (lane >= n_fin && lane < kMaxK) sh.pool_cnt[cur * kMaxK + lane] = 0;
                __syncwarp();
            } else if (mode == 4) {
                n_fin = t_nfin; covered = t_cov;                          // the memo's answer is in the slot's offer list already
            } else {
            if (cnt > 0 && mode == 1) {
                // one warp saw the whole node: its list plus the closing run (last boundary to the end) is the answer
                TopK tk;
                int fb, lb;
                warp_scan_span(lcp, d, lo, hi, K, lane, tk, fb, lb, &sh.thr_shared);
                if (lb >= 0) topk_insert(tk, K, hi - lb, lb);
                n_fin = tk.n;
                if (lane == 0) {
#pragma unroll
                    for (int i = 0; i < kMaxK; ++i) { sh.fin_cnt[i] = tk.cnt[i]; sh.fin_start[i] = tk.start[i]; }
                }
            } else if (cnt > 0) {
                const int nw = kWarps;
                __syncwarp();
                // runs that cross span edges: span w's first boundary closes the run opened by the last boundary before it
                const int wf = lane < nw ? sh.w_first[lane] : -1;
                const int wl = lane < nw ? sh.w_last[lane] : -1;
                int incl = wl;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int y = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl = max(incl, y);
                }
                int carry = __shfl_up_sync(0xffffffffu, incl, 1);
                if (lane == 0) carry = -1;
                const int last_all = __shfl_sync(0xffffffffu, incl, 31);
                int st_c = 0, st_s = 0;
                if (wf >= 0 && carry >= 0) { st_c = wf - carry; st_s = carry; }
                if (lane == 31 && last_all >= 0) { st_c = hi - last_all; st_s = last_all; }      // the closing run
                sh.st_cnt[lane] = st_c; sh.st_start[lane] = st_s;
                __syncwarp();
                // the K best of all candidates under (count desc, start asc), one warp arg-max per winner
                int* wc = &sh.w_cnt[0][0];
                int* ws = &sh.w_start[0][0];
                for (int r = 0; r < K; ++r) {
                    int xc = 0, xs = 0, xsrc = -1;
                    for (int i = lane; i < nw * kMaxK; i += 32) {
                        const int c = wc[i], st = ws[i];
                        if (c > xc || (c == xc && c > 0 && st < xs)) { xc = c; xs = st; xsrc = i; }
                    }
                    {
                        const int c = sh.st_cnt[lane], st = sh.st_start[lane];
                        if (c > xc || (c == xc && c > 0 && st < xs)) { xc = c; xs = st; xsrc = 0x1000 + lane; }
                    }
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const int oc = __shfl_xor_sync(0xffffffffu, xc, o), os = __shfl_xor_sync(0xffffffffu, xs, o);
                        const int osrc = __shfl_xor_sync(0xffffffffu, xsrc, o);
                        if (oc > xc || (oc == xc && oc > 0 && os < xs)) { xc = oc; xs = os; xsrc = osrc; }
                    }
                    if (xc <= 0) break;                                  // uniform: no candidate left
                    if (lane == 0) {
                        sh.fin_cnt[n_fin] = xc; sh.fin_start[n_fin] = xs;
                        if (xsrc >= 0x1000) sh.st_cnt[xsrc - 0x1000] = 0; else wc[xsrc] = 0;
                    }
                    ++n_fin;
                    __syncwarp();
                }
            }
            __syncwarp();
            // suffixes accounted for by the runs found
            covered = __reduce_add_sync(0xffffffffu, lane < n_fin ? sh.fin_cnt[lane] : 0);
            if (sh.long_runs_only && n_fin < K && covered < cnt) {       // uniform: fewer than k long runs and more runs exist
                __syncwarp();
                if (lane == 0) { sh.long_runs_only = 0; sh.thr_shared = 0; }
                if (mode == 1) { __syncwarp(); continue; }               // warp 0 scans it again itself
                break;
            }
            // tokens of the winners, one lane each
            if (lane < n_fin) sh.fin_tok[lane] = corpus[(int64_t)sa[sh.fin_start[lane]] + d];
            __syncwarp();
            if (t_memo_slot >= 0) {
                // claim the free entry and write the payload (another CTA may be doing the same for the same node:
                // whoever loses the claim just goes on)
                int32_t* en = memo + (size_t)t_memo_slot * kMemoInts;
                const unsigned long long key = ((unsigned long long)(unsigned)(t_full_lo + 1) << 16) | ((unsigned long long)d << 8) | (unsigned)K;
                int won = 0;
                if (lane == 0) won = atomicCAS((unsigned long long*)en, 0ull, key) == 0ull;
                won = __shfl_sync(0xffffffffu, won, 0);
                if (won) {
                    if (lane < n_fin) {                                  // counts are positive; starts and tokens get 1 added
                        en[4 + lane] = sh.fin_cnt[lane];
                        en[12 + lane] = sh.fin_start[lane] + 1;
                        en[20 + lane] = sh.fin_tok[lane] + 1;
                    }
                    if (lane == 0) en[3] = n_fin + 1;
                }
            }
            // the winners become offers, one lane each, rank = lane: count(child) * den >= num * count(parent) when a
            // threshold is set (an offer that fails it is written as retired)
            if (lane < kMaxK) {
                const int my_cnt = lane < n_fin ? sh.fin_cnt[lane] : 0;
                const bool keep = prob_num == 0 || (long long)my_cnt * prob_den >= (long long)prob_num * t_full_cnt;
                const int at = cur * kMaxK + lane;
                sh.pool_cnt[at] = keep ? my_cnt : 0;
                if (lane < n_fin) { sh.pool_tok[at] = sh.fin_tok[lane]; sh.pool_lo[at] = sh.fin_start[lane]; }
            }
            }   // a scanned node
            // ---- chain shortcut ----
            // If every occurrence of this node continues with the same token, that child has the node's own count; when
            // no pooled offer reaches that count it is the strict best and becomes the next slot, and the same holds for
            // its own single child, and so on for as long as the first and the last suffix of the interval agree (their
            // common prefix is the common prefix of the whole interval).  All those slots are emitted at once; the offer
            // written above is simply not counted in.
            if (n_fin == 1 && covered == t_full_cnt) {
                const int pmax = __reduce_max_sync(0xffffffffu, max(head0, head1));
                const int c = t_full_cnt, flo = t_full_lo, j0 = n_nodes, room = n_cap - j0;
                if (pmax < c && room > 0) {
                    const int64_t s_first = sa[flo], s_last = sa[flo + c - 1];
                    const int tf = lane < room ? corpus[s_first + d + lane] : -1;
                    const int tl = lane < room ? corpus[s_last + d + lane] : -2;
                    const unsigned eq = __ballot_sync(0xffffffffu, tf >= 0 && tf == tl);
                    const int len = eq == 0xffffffffu ? 32 : __ffs(~eq) - 1;     // leading lanes that agree (>= 1 here)
                    if (len >= 1) {
                        if (lane < len) {
                            o_ids[j0 + lane] = tf;
                            o_par[j0 + lane] = j0 + lane - 1;                    // j0 - 1 is this node (the newest slot)
                            if (o_cnt) o_cnt[j0 + lane] = c;
                            sh.slot_depth[j0 + lane] = d + 1 + lane;
                        }
                        n_nodes = j0 + len;
                        t_mode = 0;
                        if (lane == 0) { sh.n_nodes = n_nodes; sh.mode = 0; }
                        if (n_nodes < n_cap) publish(n_nodes - 1, flo, c, d + len);
                        mode = t_mode;
                        if (mode == 1 || mode == 3 || mode == 4) continue;
                        break;
                    }
                }
            }
            // the list of this slot is in place: its owner picks up the head
            __syncwarp();
            if (lane == (cur & 31)) {
                const int h = sh.pool_cnt[cur * kMaxK];
                if (cur < 32) { head0 = h; cur0 = 0; } else { head1 = h; cur1 = 0; }
            }
            __syncwarp();
            }   // mode != 6
            // ---- take the best offer: count desc, parent slot asc, token asc ----
            // Offers that tie with the best one on the count follow it in exactly this order whatever their own
            // continuations are (a continuation's count is not larger and its parent slot is newer), so all of them, up to
            // one per warp, become slots now; if they are small nodes they are expanded together in the next round.
            int n_items = 0, batch_c = 0, j = 0, slo = 0, depth = 0;
            while (true) {
                const int c_best = __reduce_max_sync(0xffffffffu, max(head0, head1));
                if (c_best <= 0 || (n_items > 0 && c_best != batch_c)) break;
                // among the lists whose head has that count the smallest slot wins; its cursor rides along
                const int mine = head0 == c_best ? (lane * kMaxK + cur0) : head1 == c_best ? ((lane + 32) * kMaxK + cur1) : 0x7fffffff;
                const int bi = __reduce_min_sync(0xffffffffu, mine);     // parent slot * kMaxK + rank = where the offer sits
                const int bp = bi / kMaxK;
                j = n_nodes;
                slo = sh.pool_lo[bi];
                depth = sh.slot_depth[bp] + 1;                           // parents were made in earlier rounds
                if (lane == (bp & 31)) {                                 // the list's owner emits the slot and moves to the next offer
                    o_ids[j] = sh.pool_tok[bi]; o_par[j] = bp;
                    if (o_cnt) o_cnt[j] = c_best;
                    sh.slot_depth[j] = depth;
                    sh.it_slot[n_items] = j; sh.it_lo[n_items] = slo; sh.it_cnt[n_items] = c_best; sh.it_depth[n_items] = depth;
                    const int nr = (bi & (kMaxK - 1)) + 1;
                    const int nh = nr < kMaxK ? sh.pool_cnt[bi + 1] : 0;
                    if (bp < 32) { cur0 = nr; head0 = nh; } else { cur1 = nr; head1 = nh; }
                }
                __syncwarp();
                ++n_nodes;
                batch_c = c_best;
                ++n_items;
                if (n_nodes >= n_cap) { n_items = -1; break; }         // the budget is used up: nothing is expanded any more
                if (c_best > 32 || n_items == kWarps) break;            // large nodes go one at a time
            }
            if (lane == 0) sh.n_nodes = n_nodes;
            __syncwarp();
            // what the next round does
            if (n_items <= 0) {
                t_mode = 0;
                if (lane == 0) sh.mode = 0;
            } else if (n_items == 1) {
                publish(j, slo, batch_c, depth);
            } else {
                t_mode = 6;
                if (lane == 0) { sh.n_items = n_items; sh.mode = 6; }
            }
            mode = t_mode;
            if (mode != 1 && mode != 3 && mode != 4) break;               // done, or the next turn needs the other warps
            }
        }
    }
    const int n = sh.n_nodes;
    if (tid == 0) num_nodes[row] = n;
    for (int j = n + tid; j < N; j += kThreads) {
        o_ids[j] = -1; o_par[j] = -1;
        if (o_cnt) o_cnt[j] = 0;
    }
}

// Candidate arrays of the scored draft, all int32, in the caller's workspace.
struct CandArrays {
    int32_t *len, *match_len, *num_nodes, *ids, *parent, *count;
};
__host__ __device__ inline CandArrays cand_layout(void* base, size_t rows, int N) {
    CandArrays c;
    int32_t* p = (int32_t*)base;
    c.len = p; p += rows;
    c.match_len = p; p += rows;
    c.num_nodes = p; p += rows;
    c.ids = p; p += rows * N;
    c.parent = p; p += rows * N;
    c.count = p;
    return c;
}

// Picks, per request, the candidate tree with the largest score = (sum of the counts of slots 1..) / (count of the
// root), compared exactly by cross-multiplication; equal scores go to the longer suffix (the smaller candidate index).
// One warp per request, one lane per candidate.
__global__ void __launch_bounds__(256)
war_draft_select_kernel(CandArrays ca, int B, int C, int N, int32_t* __restrict__ match_len, int32_t* __restrict__ used_len,
                        int32_t* __restrict__ num_nodes, int32_t* __restrict__ ids, int32_t* __restrict__ parent,
                        int32_t* __restrict__ count) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (b >= B) return;
    const size_t row = (size_t)b * C + lane;
    int len = -1, n = 0, den = 0, best = lane;
    long long num = 0;
    if (lane < C) {
        len = ca.len[row];
        if (len >= 0) {
            n = ca.num_nodes[row];
            den = n > 0 ? ca.count[row * N] : 0;
            for (int j = 1; j < n; ++j) num += ca.count[row * N + j];
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int o_len = __shfl_xor_sync(0xffffffffu, len, o), o_den = __shfl_xor_sync(0xffffffffu, den, o);
        const int o_best = __shfl_xor_sync(0xffffffffu, best, o);
        const long long o_num = __shfl_xor_sync(0xffffffffu, num, o);
        bool take;
        if (o_len < 0) take = false;
        else if (len < 0) take = true;
        else {
            // o_num / o_den against num / den by 128-bit products (counts may need 31 bits, sums 37)
            const unsigned long long l_hi = __umul64hi((unsigned long long)o_num, (unsigned long long)den), l_lo = (unsigned long long)o_num * (unsigned long long)den;
            const unsigned long long r_hi = __umul64hi((unsigned long long)num, (unsigned long long)o_den), r_lo = (unsigned long long)num * (unsigned long long)o_den;
            const bool gt = l_hi > r_hi || (l_hi == r_hi && l_lo > r_lo), eq = l_hi == r_hi && l_lo == r_lo;
            take = gt || (eq && o_best < best);
        }
        if (take) { len = o_len; den = o_den; num = o_num; best = o_best; }
    }
    // every lane holds the winner (candidate 0 is always valid)
    const size_t win = (size_t)b * C + best;
    const int wn = ca.num_nodes[win];
    if (lane == 0) { match_len[b] = ca.match_len[(size_t)b * C]; used_len[b] = max(len, 0); num_nodes[b] = wn; }
    for (int j = lane; j < N; j += 32) {
        ids[(size_t)b * N + j] = ca.ids[win * N + j];
        parent[(size_t)b * N + j] = ca.parent[win * N + j];
        if (count) count[(size_t)b * N + j] = ca.count[win * N + j];
    }
}

war_status_t launch_draft(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len, const war_draft_params_t* p,
                          int n_cand, int32_t* match_len, int32_t* num_nodes, int32_t* ids, int32_t* parent, int32_t* count,
                          int32_t* cand_len, cudaStream_t stream) {
    static int sm_count[64] = {0};
    const int dev = ix->device;
    if (dev < 0 || dev >= 64) return WAR_ERR_INVALID_ARG;
    if (!sm_count[dev]) WAR_CUDA_TRY(cudaDeviceGetAttribute(&sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
    const dim3 grid(p->B, n_cand);
    const int fac_den = p->spec_factor_num > 0 ? p->spec_factor_den : 1, prob_den = p->min_prob_num > 0 ? p->min_prob_den : 1;
    if ((long long)p->B * n_cand <= sm_count[dev])
        war_draft_kernel<1><<<grid, kThreads, 0, stream>>>(ix->corpus, ix->d_view, ix->vocab, d_tail, d_tail_len,
                                                          p->B, p->P, p->N, p->topk, p->min_match, p->spec_batch_limit, p->spec_factor_num,
                                                          fac_den, p->min_prob_num, prob_den, match_len, num_nodes, ids, parent, count, cand_len);
    else
        war_draft_kernel<2><<<grid, kThreads, 0, stream>>>(ix->corpus, ix->d_view, ix->vocab, d_tail, d_tail_len,
                                                          p->B, p->P, p->N, p->topk, p->min_match, p->spec_batch_limit, p->spec_factor_num,
                                                          fac_den, p->min_prob_num, prob_den, match_len, num_nodes, ids, parent, count, cand_len);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}

bool draft_params_ok(const war_index_t* ix, const war_draft_params_t* p) {
    if (p->B < 0 || p->P < 1 || p->P > kMaxP || p->N < 1 || p->N > kMaxN || p->topk < 1 || p->topk > kMaxK || p->min_match < 0 ||
        p->spec_batch_limit < 0 || p->spec_factor_num < 0 || (p->spec_factor_num > 0 && p->spec_factor_den < 1) ||
        p->min_prob_num < 0 || (p->min_prob_num > 0 && (p->min_prob_den < 1 || p->min_prob_num > p->min_prob_den)))
        return false;
    return p->P + p->N <= ix->max_depth;                            // else the index is not ordered deep enough
}

}  // namespace

extern "C" size_t war_draft_scored_workspace_bytes(const war_draft_params_t* p, int32_t n_lengths) {
    if (!p || p->B < 0 || p->N < 1 || p->N > kMaxN || n_lengths < 1 || n_lengths > kMaxP) return 0;
    const size_t rows = (size_t)p->B * n_lengths;
    return sizeof(int32_t) * (3 * rows + 3 * rows * p->N) + 256;
}

extern "C" war_status_t war_draft_scored(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len,
                                         const war_draft_params_t* p, int32_t n_lengths, void* d_workspace,
                                         int32_t* d_match_len, int32_t* d_used_len, int32_t* d_num_nodes, int32_t* d_ids,
                                         int32_t* d_parent, int32_t* d_count, war_stream_t stream) {
    if (!ix || !p) return WAR_ERR_INVALID_ARG;
    if (!draft_params_ok(ix, p) || n_lengths < 1 || n_lengths > kMaxP) return WAR_ERR_INVALID_ARG;
    if (p->B == 0) return WAR_OK;
    if (!d_tail || !d_tail_len || !d_workspace || !d_match_len || !d_used_len || !d_num_nodes || !d_ids || !d_parent)
        return WAR_ERR_INVALID_ARG;
    const CandArrays ca = cand_layout(d_workspace, (size_t)p->B * n_lengths, p->N);
    const war_status_t st = launch_draft(ix, d_tail, d_tail_len, p, n_lengths, ca.match_len, ca.num_nodes, ca.ids, ca.parent, ca.count,
                                         ca.len, stream);
    if (st != WAR_OK) return st;
    war_draft_select_kernel<<<(p->B + 7) / 8, 256, 0, stream>>>(ca, p->B, n_lengths, p->N, d_match_len, d_used_len, d_num_nodes,
                                                              d_ids, d_parent, d_count);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}

extern "C" war_status_t war_draft(const war_index_t* ix, const int32_t* d_tail, const int32_t* d_tail_len,
                                  const war_draft_params_t* p, int32_t* d_match_len, int32_t* d_num_nodes,
                                  int32_t* d_ids, int32_t* d_parent, int32_t* d_count, war_stream_t stream) {
    if (!ix || !p) return WAR_ERR_INVALID_ARG;
    if (!draft_params_ok(ix, p)) return WAR_ERR_INVALID_ARG;
    if (p->B == 0) return WAR_OK;
    if (!d_tail || !d_tail_len || !d_match_len || !d_num_nodes || !d_ids || !d_parent) return WAR_ERR_INVALID_ARG;
    return launch_draft(ix, d_tail, d_tail_len, p, 1, d_match_len, d_num_nodes, d_ids, d_parent, d_count, nullptr, stream);
}
