// Trajectory cache: suffix array + capped LCP + first-token buckets over the separator-joined corpus.
//
// Only ordering to depth max_depth (<= 128) is ever needed by the draft kernel (it compares at most P pattern
// tokens and descends at most N-1 further), so prefix doubling stops after ceil(log2(max_depth)) rounds.
// Round r sorts 64-bit keys (rank of the first 2^r tokens, rank of the next 2^r tokens) with a device radix
// sort and re-ranks by adjacent difference + scan; suffixes whose rank is already unique drop out of later rounds.
// Suffixes that still tie after the last round keep the order the stable sort left them in; no output of the
// library depends on that order.
#include <cub/cub.cuh>
#include <cstring>
#include <new>
#include "war_common.cuh"
#include "war_index.cuh"

namespace {

constexpr int kThreads = 256;

struct MaxOp {
    __device__ __forceinline__ uint32_t operator()(uint32_t a, uint32_t b) const { return a > b ? a : b; }
};

// corpus[dst_base + off[t] + t + i] = tokens[off[t] + i]; separator -(t0 + t + 1) after each trajectory.
// A token id outside [0, vocab) raises *bad (such ids would collide with separators or overflow the sort keys).
__global__ void scatter_corpus_kernel(const int32_t* __restrict__ tokens, const int64_t* __restrict__ off, int T,
                                      int t0, int64_t dst_base, int32_t* __restrict__ corpus, int64_t n_out, int vocab,
                                      int* __restrict__ bad, int* __restrict__ status_word) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_out) return;
    // trajectory t covers output positions [off[t] + t, off[t+1] + t]; the last one is its separator
    int lo = 0, hi = T - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (off[mid] + mid <= i) lo = mid; else hi = mid - 1;
    }
    const int t = lo;
    const int64_t local = i - (off[t] + t);
    const int64_t len = off[t + 1] - off[t];
    int32_t v = -(t0 + t + 1);
    if (local < len) {
        v = tokens[off[t] + local];
        if (v < 0 || v >= vocab) {
            if (bad) *bad = 1;
            // stream-ordered append: nobody reads a flag back, so the token becomes an end-of-trajectory mark (it
            // matches nothing and nothing continues into it) and the problem goes to the device status word
            if (status_word) { war_set_device_status(status_word, WAR_ERR_INVALID_ARG); v = -(t0 + t + 1); }
        }
    }
    corpus[dst_base + i] = v;
}

// first-round key: separators (negative, unique) below every token
__global__ void init_keys_kernel(const int32_t* __restrict__ corpus, int64_t M, int T, uint32_t* __restrict__ key,
                                 int32_t* __restrict__ sa) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    key[i] = (uint32_t)(corpus[i] + T);
    sa[i] = (int32_t)i;
}

__global__ void flag32_kernel(const uint32_t* __restrict__ key, int64_t M, uint32_t* __restrict__ flag) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    flag[i] = (i > 0 && key[i] != key[i - 1]) ? (uint32_t)i : 0u;
}

// rank[sa[i]] = index of the first suffix of i's group
__global__ void scatter_rank_kernel(const int32_t* __restrict__ sa, const uint32_t* __restrict__ group_start, int64_t M,
                                    uint32_t* __restrict__ rank) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    rank[sa[i]] = group_start[i];
}

__global__ void lcp_kernel(const int32_t* __restrict__ corpus, const int32_t* __restrict__ sa, int64_t M, int max_depth,
                           uint8_t* __restrict__ lcp) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    int l = 0;
    if (i > 0) {
        const int64_t a = sa[i - 1], b = sa[i];
        // separators are unique, so the comparison stops at the first one; the last corpus entry is a separator
        while (l < max_depth && a + l < M && b + l < M && corpus[a + l] == corpus[b + l]) ++l;
    }
    lcp[i] = (uint8_t)l;
}

struct Scratch {
    void* p = nullptr;
    ~Scratch() { if (p) cudaFree(p); }
};

inline dim3 grid_for(int64_t n) { return dim3((unsigned)((n + kThreads - 1) / kThreads)); }

// ---- prefix doubling over the suffixes that are still tied ---------------------------------------
// After a round, a suffix whose rank is unique is final.  Later rounds only touch the slots of groups that still
// hold two or more suffixes (`act`, ascending slot numbers): their (rank, rank at +h) keys are sorted on their own
// and written back into the same slots, because a group occupies a contiguous slot range and the key's upper word
// (the group's rank) keeps groups in slot order.

__global__ void active_keys_kernel(const int32_t* __restrict__ act, const int32_t* __restrict__ sa, const uint32_t* __restrict__ rank,
                                   int64_t n, int64_t h, int64_t m, uint64_t* __restrict__ key, int32_t* __restrict__ val) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= m) return;
    const int64_t s = sa[act[a]];
    const uint64_t hi = rank[s];
    const uint64_t lo = (s + h < n) ? (uint64_t)rank[s + h] + 1u : 0u;
    key[a] = (hi << 32) | lo;
    val[a] = (int32_t)s;
}

// writes the sorted suffixes back into their slots; head[a] = slot number if a starts a new (sub)group, else 0
__global__ void active_writeback_kernel(const int32_t* __restrict__ act, const uint64_t* __restrict__ key, const int32_t* __restrict__ val,
                                        int64_t m, int32_t* __restrict__ sa, uint32_t* __restrict__ head) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= m) return;
    sa[act[a]] = val[a];
    head[a] = (a == 0 || key[a] != key[a - 1]) ? (uint32_t)act[a] : 0u;
}

__global__ void active_rank_kernel(const int32_t* __restrict__ val, const uint32_t* __restrict__ grp, int64_t m, uint32_t* __restrict__ rank) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a < m) rank[val[a]] = grp[a];
}

// keep[a] = 1 unless the suffix in slot act[a] is alone in its group (grp = slot of the group's first suffix)
__global__ void active_keep_kernel(const int32_t* __restrict__ act, const uint32_t* __restrict__ grp, int64_t m, uint8_t* __restrict__ keep) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= m) return;
    const bool is_head = grp[a] == (uint32_t)act[a];
    const bool next_is_head = a + 1 == m || grp[a + 1] == (uint32_t)act[a + 1];
    keep[a] = (is_head && next_is_head) ? 0 : 1;
}

__global__ void iota_kernel(int32_t* __restrict__ x, int64_t n) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) x[i] = (int32_t)i;
}

// Sorts the n suffixes of `corpus[0 .. n)` (a run of whole trajectories, each ending in its separator) to depth
// max_depth by prefix doubling and writes their start positions, relative to `corpus`, to out_sa (device, n entries).
// T_total shifts the symbols so that every separator -(t+1), t < T_total, maps to a non-negative key.
war_status_t sort_suffixes(const int32_t* corpus, int64_t n64, int T_total, int vocab, int max_depth, int32_t* out_sa,
                           cudaStream_t s) {
    const int n = (int)n64;
    size_t t_sort64 = 0, t_sort32 = 0, t_scan = 0, t_sel = 0;
    {
        cub::DoubleBuffer<uint64_t> k64(nullptr, nullptr);
        cub::DoubleBuffer<uint32_t> k32(nullptr, nullptr);
        cub::DoubleBuffer<int32_t> v(nullptr, nullptr);
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, t_sort64, k64, v, n, 0, 64, s));
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(nullptr, t_sort32, k32, v, n, 0, 32, s));
        WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, t_scan, (uint32_t*)nullptr, (uint32_t*)nullptr, MaxOp(), n, s));
        WAR_CUDA_TRY(cub::DeviceSelect::Flagged(nullptr, t_sel, (int32_t*)nullptr, (uint8_t*)nullptr, (int32_t*)nullptr, (int*)nullptr, n, s));
    }
    size_t temp_bytes = t_sort64;
    if (t_sort32 > temp_bytes) temp_bytes = t_sort32;
    if (t_scan > temp_bytes) temp_bytes = t_scan;
    if (t_sel > temp_bytes) temp_bytes = t_sel;
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t b_key = align(sizeof(uint64_t) * n64), b_i32 = align(sizeof(int32_t) * n64), b_u8 = align((size_t)n64);
    // key x2, val x2, rank, head/group, act x2, keep, one counter, cub temp
    const size_t total = 2 * b_key + 2 * b_i32 + 2 * b_i32 + 2 * b_i32 + b_u8 + 256 + align(temp_bytes);
    Scratch scratch;
    WAR_CUDA_TRY(cudaMalloc(&scratch.p, total));
    char* at = (char*)scratch.p;
    uint64_t* key_a = (uint64_t*)at; at += b_key;
    uint64_t* key_b = (uint64_t*)at; at += b_key;
    int32_t* val_a = (int32_t*)at; at += b_i32;
    int32_t* val_b = (int32_t*)at; at += b_i32;
    uint32_t* rank = (uint32_t*)at; at += b_i32;
    uint32_t* head = (uint32_t*)at; at += b_i32;
    int32_t* act_a = (int32_t*)at; at += b_i32;
    int32_t* act_b = (int32_t*)at; at += b_i32;
    uint8_t* keep = (uint8_t*)at; at += b_u8;
    int* d_count = (int*)at; at += 256;
    void* temp = at;

    int sym_bits = 1;
    while (((int64_t)1 << sym_bits) < (int64_t)vocab + T_total) ++sym_bits;
    int pos_bits = 1;
    while (((int64_t)1 << pos_bits) < n64 + 1) ++pos_bits;

    // round 0: order everything by the first token; out_sa holds the slots from here on
    {
        cub::DoubleBuffer<uint32_t> k32((uint32_t*)key_a, (uint32_t*)key_b);
        cub::DoubleBuffer<int32_t> val(val_a, val_b);
        init_keys_kernel<<<grid_for(n64), kThreads, 0, s>>>(corpus, n64, T_total, k32.Current(), val.Current());
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, temp_bytes, k32, val, n, 0, sym_bits, s));
        WAR_CUDA_TRY(cudaMemcpyAsync(out_sa, val.Current(), sizeof(int32_t) * n64, cudaMemcpyDeviceToDevice, s));
        flag32_kernel<<<grid_for(n64), kThreads, 0, s>>>(k32.Current(), n64, head);
        WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, head, head, MaxOp(), n, s));
        scatter_rank_kernel<<<grid_for(n64), kThreads, 0, s>>>(out_sa, head, n64, rank);
        iota_kernel<<<grid_for(n64), kThreads, 0, s>>>(act_a, n64);
        active_keep_kernel<<<grid_for(n64), kThreads, 0, s>>>(act_a, head, n64, keep);
        WAR_CUDA_TRY(cub::DeviceSelect::Flagged(temp, temp_bytes, act_a, keep, act_b, d_count, n, s));
    }
    int32_t* act = act_b;
    int32_t* act_other = act_a;
    int m = 0;
    WAR_CUDA_TRY(cudaMemcpyAsync(&m, d_count, sizeof(int), cudaMemcpyDeviceToHost, s));
    WAR_CUDA_TRY(cudaStreamSynchronize(s));
    for (int64_t h = 1; h < max_depth && m > 0; h <<= 1) {
        cub::DoubleBuffer<uint64_t> k64(key_a, key_b);
        cub::DoubleBuffer<int32_t> val(val_a, val_b);
        active_keys_kernel<<<grid_for(m), kThreads, 0, s>>>(act, out_sa, rank, n64, h, m, k64.Current(), val.Current());
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, temp_bytes, k64, val, m, 0, 32 + pos_bits, s));
        active_writeback_kernel<<<grid_for(m), kThreads, 0, s>>>(act, k64.Current(), val.Current(), m, out_sa, head);
        WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, head, head, MaxOp(), m, s));
        active_rank_kernel<<<grid_for(m), kThreads, 0, s>>>(val.Current(), head, m, rank);
        if ((h << 1) >= max_depth) break;                    // last round: nobody needs the next active list
        active_keep_kernel<<<grid_for(m), kThreads, 0, s>>>(act, head, m, keep);
        WAR_CUDA_TRY(cub::DeviceSelect::Flagged(temp, temp_bytes, act, keep, act_other, d_count, m, s));
        WAR_CUDA_TRY(cudaMemcpyAsync(&m, d_count, sizeof(int), cudaMemcpyDeviceToHost, s));
        WAR_CUDA_TRY(cudaStreamSynchronize(s));
        int32_t* tmp = act; act = act_other; act_other = tmp;
    }
    WAR_LAUNCH_CHECK();
    WAR_CUDA_TRY(cudaStreamSynchronize(s));          // the scratch is freed on return
    return WAR_OK;
}

// bucket[v] = first suffix-array index whose suffix starts with a token >= v (tokens ascend along the suffix array,
// the T separators come first); one thread per entry fills the gap between its predecessor's token and its own.
__global__ void bucket_from_sa_kernel(const int32_t* __restrict__ corpus, const int32_t* __restrict__ sa, int64_t M, int vocab,
                                      int32_t* __restrict__ bucket) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i > M) return;
    const int cur = i < M ? max(corpus[sa[i]], -1) : vocab;          // sentinel after the last suffix
    const int prev = i > 0 ? max(corpus[sa[i - 1]], -1) : -1;
    for (int v = prev + 1; v <= min(cur, vocab); ++v) bucket[v] = (int32_t)i;
}

// lcp and buckets of the shadow set from its finished suffix array; then the shadow set is published
war_status_t finish_index(war_index* ix, cudaStream_t s) {
    const int64_t M = ix->M;
    war_index_arrays& a = ix->shadow();
    lcp_kernel<<<grid_for(M), kThreads, 0, s>>>(ix->corpus, a.sa, M, ix->max_depth, a.lcp);
    bucket_from_sa_kernel<<<grid_for(M + 1), kThreads, 0, s>>>(ix->corpus, a.sa, M, ix->vocab, a.bucket);
    WAR_LAUNCH_CHECK();
    WAR_CUDA_TRY(cudaMemsetAsync(a.memo, 0, sizeof(int32_t) * kMemoEntries * kMemoInts, s));   // it described another suffix array
    WAR_CUDA_TRY(ix->publish(s));
    return WAR_OK;
}

// (Re)builds sa / lcp / bucket from ix->corpus[0 .. M) in the shadow set and publishes it.
war_status_t rebuild(war_index* ix, cudaStream_t s) {
    const int64_t M = ix->M;
    if (M == 0) {
        WAR_CUDA_TRY(cudaMemsetAsync(ix->shadow().bucket, 0, sizeof(int32_t) * (ix->vocab + 1), s));
        WAR_CUDA_TRY(ix->publish(s));
        return WAR_OK;
    }
    const war_status_t st = sort_suffixes(ix->corpus, M, ix->T, ix->vocab, ix->max_depth, ix->shadow().sa, s);
    if (st != WAR_OK) return st;
    return finish_index(ix, s);
}

// ---- incremental append -------------------------------------------------------------------------
// Separators isolate trajectories, so appending never changes the relative order of the old suffixes.  The new
// suffixes are sorted among themselves, each finds how many old suffixes precede it (binary search inside its first
// token's old bucket, to the depth the index is ordered to), and the two sorted lists are merged by scatter.

// pos[j] = number of old suffixes that sort before new suffix j (lower bound; equal-to-depth ties go after it)
__global__ void insert_pos_kernel(const int32_t* __restrict__ corpus, const int32_t* __restrict__ sa_old,
                                  const int32_t* __restrict__ bucket_old, const int32_t* __restrict__ new_sa, int64_t m, int64_t M_old,
                                  int vocab, int depth, uint32_t* __restrict__ pos) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= m) return;
    const int64_t p = M_old + new_sa[j];
    const int c0 = corpus[p];
    if (c0 < 0 || c0 >= vocab) { pos[j] = 0u; return; }     // new separators are smaller than every old entry
    int a = bucket_old[c0], z = bucket_old[c0 + 1];
    int ma = 1, mz = 1;                                     // tokens known equal at the current ends (bucket: token 0)
    while (a < z) {
        const int mid = a + ((z - a) >> 1);
        const int64_t q = sa_old[mid];
        int t = min(ma, mz);
        int cmp = 0;                                        // sign of (old suffix - new suffix)
        for (; t < depth; ++t) {
            const int x = corpus[q + t], y = corpus[p + t];
            if (x != y) { cmp = x < y ? -1 : 1; break; }
        }
        if (cmp < 0) { a = mid + 1; ma = t; } else { z = mid; mz = t; }
    }
    pos[j] = (uint32_t)a;
}

__global__ void count_pos_kernel(const uint32_t* __restrict__ pos, int64_t m, uint32_t* __restrict__ add) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < m) atomicAdd(&add[pos[j]], 1u);
}

// old suffix i moves behind the new suffixes that were inserted at or before it
__global__ void scatter_old_kernel(const int32_t* __restrict__ sa_old, const uint32_t* __restrict__ shift, int64_t M_old,
                                   int32_t* __restrict__ sa_out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < M_old) sa_out[i + shift[i]] = sa_old[i];
}

__global__ void scatter_new_kernel(const int32_t* __restrict__ new_sa, const uint32_t* __restrict__ pos, int64_t m, int64_t M_old,
                                   int32_t* __restrict__ sa_out) {
    const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < m) sa_out[(int64_t)pos[j] + j] = (int32_t)(M_old + new_sa[j]);
}

struct SumOp {
    __device__ __forceinline__ uint32_t operator()(uint32_t a, uint32_t b) const { return a + b; }
};

war_status_t merge_new_suffixes(war_index* ix, int64_t M_old, cudaStream_t s) {
    const int64_t M = ix->M, m = M - M_old;
    const war_index_arrays old = ix->published();
    int32_t* sa_out = ix->shadow().sa;
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    size_t temp_scan = 0, temp_scan2 = 0;
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, temp_scan, (uint32_t*)nullptr, (uint32_t*)nullptr, MaxOp(), (int)m, s));
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, temp_scan2, (uint32_t*)nullptr, (uint32_t*)nullptr, SumOp(), (int)(M_old + 1), s));
    size_t temp_bytes = temp_scan > temp_scan2 ? temp_scan : temp_scan2;
    const size_t b_new = align(sizeof(int32_t) * m), b_pos = align(sizeof(uint32_t) * m), b_add = align(sizeof(uint32_t) * (M_old + 1));
    Scratch scratch;
    WAR_CUDA_TRY(cudaMalloc(&scratch.p, b_new + b_pos + b_add + align(temp_bytes)));
    char* at = (char*)scratch.p;
    int32_t* new_sa = (int32_t*)at; at += b_new;
    uint32_t* pos = (uint32_t*)at; at += b_pos;
    uint32_t* add = (uint32_t*)at; at += b_add;
    void* temp = at;

    war_status_t st = sort_suffixes(ix->corpus + M_old, m, ix->T, ix->vocab, ix->max_depth, new_sa, s);
    if (st != WAR_OK) return st;
    insert_pos_kernel<<<grid_for(m), kThreads, 0, s>>>(ix->corpus, old.sa, old.bucket, new_sa, m, M_old, ix->vocab, ix->max_depth, pos);
    // positions must not decrease along the sorted new suffixes (they cannot, up to ties at full depth): enforce it
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, pos, pos, MaxOp(), (int)m, s));
    WAR_CUDA_TRY(cudaMemsetAsync(add, 0, b_add, s));
    count_pos_kernel<<<grid_for(m), kThreads, 0, s>>>(pos, m, add);
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, add, add, SumOp(), (int)(M_old + 1), s));
    scatter_old_kernel<<<grid_for(M_old), kThreads, 0, s>>>(old.sa, add, M_old, sa_out);
    scatter_new_kernel<<<grid_for(m), kThreads, 0, s>>>(new_sa, pos, m, M_old, sa_out);
    WAR_LAUNCH_CHECK();
    st = finish_index(ix, s);
    return st;
}

war_status_t check_offsets(const int64_t* h_offsets, int32_t T) {
    if (T < 0) return WAR_ERR_INVALID_ARG;
    if (T > 0 && !h_offsets) return WAR_ERR_INVALID_ARG;
    for (int t = 0; t < T; ++t)
        if (h_offsets[t + 1] < h_offsets[t]) return WAR_ERR_INVALID_ARG;
    if (T > 0 && h_offsets[0] < 0) return WAR_ERR_INVALID_ARG;
    return WAR_OK;
}

// Adds T trajectories (device tokens, host offsets) behind the current corpus content.
war_status_t add_trajectories(war_index* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T, cudaStream_t s) {
    if (T == 0) return WAR_OK;
    const int64_t n_tok = h_offsets[T] - h_offsets[0];
    const int64_t n_out = n_tok + T;
    if (ix->M + n_out > ix->capacity || ix->M + n_out >= ((int64_t)1 << 31) - 256 || (int64_t)ix->T + T >= ((int64_t)1 << 30))
        return WAR_ERR_CAPACITY;
    if (n_tok > 0 && !d_tokens) return WAR_ERR_INVALID_ARG;
    // offsets relative to the first trajectory of this batch
    int64_t* rel = new (std::nothrow) int64_t[T + 1];
    if (!rel) return WAR_ERR_OOM;
    for (int t = 0; t <= T; ++t) rel[t] = h_offsets[t] - h_offsets[0];
    Scratch off;                                             // offsets, then one int: the bad-token flag
    int bad = 0;
    cudaError_t e = cudaMalloc(&off.p, sizeof(int64_t) * (T + 2));
    int* d_bad = e == cudaSuccess ? (int*)((int64_t*)off.p + (T + 1)) : nullptr;
    if (e == cudaSuccess) e = cudaMemcpyAsync(off.p, rel, sizeof(int64_t) * (T + 1), cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(d_bad, 0, sizeof(int), s);
    if (e == cudaSuccess) {
        scatter_corpus_kernel<<<grid_for(n_out), kThreads, 0, s>>>(d_tokens + h_offsets[0], (const int64_t*)off.p, T, ix->T,
                                                                  ix->M, ix->corpus, n_out, ix->vocab, d_bad, nullptr);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    delete[] rel;
    if (e != cudaSuccess) { (void)cudaGetLastError(); return e == cudaErrorMemoryAllocation ? WAR_ERR_OOM : WAR_ERR_CUDA; }
    if (bad) return WAR_ERR_INVALID_ARG;                     // nothing was committed: M and T are unchanged
    try {
        for (int t = 1; t <= T; ++t) ix->bounds.push_back(ix->M + (h_offsets[t] - h_offsets[0]) + t);
    } catch (...) {
        ix->bounds.resize((size_t)ix->T + 1);
        return WAR_ERR_OOM;
    }
    ix->M += n_out;
    ix->T += T;
    return WAR_OK;
}

// ---- eviction of the oldest trajectories ----------------------------------------------------------
// Suffixes of the remaining trajectories keep their relative order (separators isolate trajectories and keep their
// own order when all of them are renumbered by the same amount), so the suffix array is filtered, not sorted again.
struct KeepFrom {
    int32_t cut;
    __device__ __forceinline__ bool operator()(const int32_t& x) const { return x >= cut; }
};

__global__ void shift_sa_kernel(int32_t* __restrict__ sa, int64_t n, int32_t cut) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) sa[i] -= cut;
}

// dst[i] = src[cut + i], separators renumbered from -(1) again
__global__ void shift_corpus_kernel(const int32_t* __restrict__ src, int64_t n, int64_t cut, int32_t n_evicted, int32_t* __restrict__ dst) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int32_t v = src[cut + i];
    dst[i] = v < 0 ? v + n_evicted : v;
}

war_status_t evict_oldest(war_index* ix, int32_t n, cudaStream_t s) {
    const int64_t cut = ix->bounds[(size_t)n], M_old = ix->M, M = M_old - cut;
    const war_index_arrays old = ix->published();
    if (M > 0) {
        size_t temp_bytes = 0;
        WAR_CUDA_TRY(cub::DeviceSelect::If(nullptr, temp_bytes, (int32_t*)nullptr, (int32_t*)nullptr, (int32_t*)nullptr, (int)M_old,
                                           KeepFrom{(int32_t)cut}, s));
        auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
        Scratch scratch;
        WAR_CUDA_TRY(cudaMalloc(&scratch.p, align(sizeof(int32_t) * M) + align(sizeof(int32_t)) + align(temp_bytes)));
        int32_t* tmp = (int32_t*)scratch.p;
        int32_t* d_n = (int32_t*)((char*)scratch.p + align(sizeof(int32_t) * M));
        void* temp = (char*)d_n + align(sizeof(int32_t));
        int32_t* sa_new = ix->shadow().sa;
        WAR_CUDA_TRY(cub::DeviceSelect::If(temp, temp_bytes, old.sa, sa_new, d_n, (int)M_old, KeepFrom{(int32_t)cut}, s));
        shift_sa_kernel<<<grid_for(M), kThreads, 0, s>>>(sa_new, M, (int32_t)cut);
        shift_corpus_kernel<<<grid_for(M), kThreads, 0, s>>>(ix->corpus, M, cut, n, tmp);
        WAR_CUDA_TRY(cudaMemcpyAsync(ix->corpus, tmp, sizeof(int32_t) * M, cudaMemcpyDeviceToDevice, s));
        WAR_LAUNCH_CHECK();
        WAR_CUDA_TRY(cudaStreamSynchronize(s));
    }
    // the vacated end reads as "no token" again (readable slack behind the last separator)
    WAR_CUDA_TRY(cudaMemsetAsync(ix->corpus + M, 0xff, sizeof(int32_t) * (size_t)(M_old - M), s));
    ix->bounds.erase(ix->bounds.begin(), ix->bounds.begin() + n);
    for (auto& b : ix->bounds) b -= cut;
    ix->M = M;
    ix->T -= n;
    if (M == 0) {
        WAR_CUDA_TRY(cudaMemsetAsync(ix->shadow().bucket, 0, sizeof(int32_t) * (ix->vocab + 1), s));
        WAR_CUDA_TRY(ix->publish(s));
        return WAR_OK;
    }
    return finish_index(ix, s);
}

// ---- stream-ordered append ----------------------------------------------------------------------------
// The same result as war_index_append, enqueued on the caller's stream without a single host synchronisation: scratch
// comes from the stream-ordered allocator, sized from what the host knows (token and trajectory counts); the prefix
// doubling runs its fixed number of rounds over all new suffixes instead of shrinking the active set by counts read
// back from the device; the publication is a one-word kernel behind everything that built the set.

__global__ void set_u32_kernel(unsigned int* p, unsigned int v) { *p = v; }

__global__ void full_keys_kernel(const int32_t* __restrict__ sa, const uint32_t* __restrict__ rank, int64_t n, int64_t h,
                                 uint64_t* __restrict__ key, int32_t* __restrict__ val) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= n) return;
    const int64_t s = sa[a];
    const uint64_t hi = rank[s];
    const uint64_t lo = (s + h < n) ? (uint64_t)rank[s + h] + 1u : 0u;
    key[a] = (hi << 32) | lo;
    val[a] = (int32_t)s;
}

// head[a] = a if slot a starts a new group, else 0 (the inclusive max scan turns it into the group's first slot)
__global__ void full_heads_kernel(const uint64_t* __restrict__ key, int64_t n, uint32_t* __restrict__ head) {
    const int64_t a = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (a >= n) return;
    head[a] = (a > 0 && key[a] != key[a - 1]) ? (uint32_t)a : 0u;
}

size_t sort_full_scratch_bytes(int64_t n64, size_t* temp_bytes_out) {
    const int n = (int)n64;
    size_t t_sort64 = 0, t_sort32 = 0, t_scan = 0;
    cub::DoubleBuffer<uint64_t> k64(nullptr, nullptr);
    cub::DoubleBuffer<uint32_t> k32(nullptr, nullptr);
    cub::DoubleBuffer<int32_t> v(nullptr, nullptr);
    cub::DeviceRadixSort::SortPairs(nullptr, t_sort64, k64, v, n, 0, 64, (cudaStream_t)0);
    cub::DeviceRadixSort::SortPairs(nullptr, t_sort32, k32, v, n, 0, 32, (cudaStream_t)0);
    cub::DeviceScan::InclusiveScan(nullptr, t_scan, (uint32_t*)nullptr, (uint32_t*)nullptr, MaxOp(), n, (cudaStream_t)0);
    size_t temp = t_sort64 > t_sort32 ? t_sort64 : t_sort32;
    if (t_scan > temp) temp = t_scan;
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    *temp_bytes_out = align(temp);
    return 2 * align(sizeof(uint64_t) * n64) + 4 * align(sizeof(int32_t) * n64) + align(temp);
}

// sort_suffixes without host round trips: every round sorts all n (rank, rank at +h) keys.  `scratch` holds
// sort_full_scratch_bytes(n) bytes.  Ties beyond max_depth keep the order of the start positions, as in sort_suffixes.
war_status_t sort_suffixes_full(const int32_t* corpus, int64_t n64, int T_total, int vocab, int max_depth, int32_t* out_sa,
                                void* scratch, cudaStream_t s) {
    const int n = (int)n64;
    size_t temp_bytes = 0;
    (void)sort_full_scratch_bytes(n64, &temp_bytes);
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t b_key = align(sizeof(uint64_t) * n64), b_i32 = align(sizeof(int32_t) * n64);
    char* at = (char*)scratch;
    uint64_t* key_a = (uint64_t*)at; at += b_key;
    uint64_t* key_b = (uint64_t*)at; at += b_key;
    int32_t* val_a = (int32_t*)at; at += b_i32;
    int32_t* val_b = (int32_t*)at; at += b_i32;
    uint32_t* rank = (uint32_t*)at; at += b_i32;
    uint32_t* head = (uint32_t*)at; at += b_i32;
    void* temp = at;
    int sym_bits = 1;
    while (((int64_t)1 << sym_bits) < (int64_t)vocab + T_total) ++sym_bits;
    int pos_bits = 1;
    while (((int64_t)1 << pos_bits) < n64 + 1) ++pos_bits;
    {
        cub::DoubleBuffer<uint32_t> k32((uint32_t*)key_a, (uint32_t*)key_b);
        cub::DoubleBuffer<int32_t> val(val_a, val_b);
        init_keys_kernel<<<grid_for(n64), kThreads, 0, s>>>(corpus, n64, T_total, k32.Current(), val.Current());
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, temp_bytes, k32, val, n, 0, sym_bits, s));
        WAR_CUDA_TRY(cudaMemcpyAsync(out_sa, val.Current(), sizeof(int32_t) * n64, cudaMemcpyDeviceToDevice, s));
        flag32_kernel<<<grid_for(n64), kThreads, 0, s>>>(k32.Current(), n64, head);
        WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, head, head, MaxOp(), n, s));
        scatter_rank_kernel<<<grid_for(n64), kThreads, 0, s>>>(out_sa, head, n64, rank);
    }
    for (int64_t h = 1; h < max_depth; h <<= 1) {
        cub::DoubleBuffer<uint64_t> k64(key_a, key_b);
        cub::DoubleBuffer<int32_t> val(val_a, val_b);
        full_keys_kernel<<<grid_for(n64), kThreads, 0, s>>>(out_sa, rank, n64, h, k64.Current(), val.Current());
        WAR_CUDA_TRY(cub::DeviceRadixSort::SortPairs(temp, temp_bytes, k64, val, n, 0, 32 + pos_bits, s));
        WAR_CUDA_TRY(cudaMemcpyAsync(out_sa, val.Current(), sizeof(int32_t) * n64, cudaMemcpyDeviceToDevice, s));
        full_heads_kernel<<<grid_for(n64), kThreads, 0, s>>>(k64.Current(), n64, head);
        WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(temp, temp_bytes, head, head, MaxOp(), n, s));
        scatter_rank_kernel<<<grid_for(n64), kThreads, 0, s>>>(out_sa, head, n64, rank);
    }
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}

struct AsyncScratch {
    void* p = nullptr;
    cudaStream_t s = nullptr;
    ~AsyncScratch() { if (p) cudaFreeAsync(p, s); }
};

// Memory freed to the stream-ordered allocator stays in its pool, so that the next update finds it without a trip to
// the driver (once per device).
void keep_pool_memory(int device) {
    static std::once_flag once[64];
    if (device < 0 || device >= 64) return;
    std::call_once(once[device], [device]() {
        cudaMemPool_t pool;
        if (cudaDeviceGetDefaultMemPool(&pool, device) == cudaSuccess) {
            unsigned long long keep = ~0ull;
            cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        }
        (void)cudaGetLastError();
    });
}

war_status_t append_async(war_index* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T, cudaStream_t s) {
    const int64_t n_tok = h_offsets[T] - h_offsets[0];
    const int64_t m = n_tok + T, M_old = ix->M, M = M_old + m;
    const int32_t T_old = ix->T;
    if (M > ix->capacity || M >= ((int64_t)1 << 31) - 256 || (int64_t)T_old + T >= ((int64_t)1 << 30)) return WAR_ERR_CAPACITY;
    if (n_tok > 0 && !d_tokens) return WAR_ERR_INVALID_ARG;
    if ((size_t)T + 1 > war_index::kStageEntries) return WAR_ERR_UNSUPPORTED;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    keep_pool_memory(ix->device);
    const bool merge = M_old > 0 && m < M_old;
    // ---- scratch, one stream-ordered allocation ----
    auto align = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const int64_t n_sort = merge ? m : M;
    size_t sort_temp = 0, temp_scan = 0, temp_scan2 = 0;
    const size_t b_sort = sort_full_scratch_bytes(n_sort, &sort_temp);
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, temp_scan, (uint32_t*)nullptr, (uint32_t*)nullptr, MaxOp(), (int)m, s));
    WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(nullptr, temp_scan2, (uint32_t*)nullptr, (uint32_t*)nullptr, SumOp(), (int)(M_old + 1), s));
    size_t b_scan = align(temp_scan > temp_scan2 ? temp_scan : temp_scan2);
    const size_t b_off = align(sizeof(int64_t) * ((size_t)T + 1)), b_new = align(sizeof(int32_t) * m), b_pos = align(sizeof(uint32_t) * m),
                 b_add = align(sizeof(uint32_t) * (M_old + 1));
    AsyncScratch scratch;
    scratch.s = s;
    WAR_CUDA_TRY(cudaMallocAsync(&scratch.p, b_off + b_sort + (merge ? b_new + b_pos + b_add + b_scan : 0), s));
    char* at = (char*)scratch.p;
    int64_t* d_off = (int64_t*)at; at += b_off;
    void* sort_scratch = at; at += b_sort;
    int32_t* new_sa = (int32_t*)at; at += merge ? b_new : 0;
    uint32_t* pos = (uint32_t*)at; at += merge ? b_pos : 0;
    uint32_t* add = (uint32_t*)at; at += merge ? b_add : 0;
    void* scan_temp = at;
    // ---- the trajectories' bounds go through pinned staging memory (its previous use has long been consumed) ----
    WAR_CUDA_TRY(cudaEventSynchronize(ix->stage_free));
    for (int t = 0; t <= T; ++t) ix->h_stage[t] = h_offsets[t] - h_offsets[0];
    WAR_CUDA_TRY(cudaMemcpyAsync(d_off, ix->h_stage, sizeof(int64_t) * ((size_t)T + 1), cudaMemcpyHostToDevice, s));
    WAR_CUDA_TRY(cudaEventRecord(ix->stage_free, s));
    scatter_corpus_kernel<<<grid_for(m), kThreads, 0, s>>>(d_tokens + h_offsets[0], d_off, T, T_old, M_old, ix->corpus, m, ix->vocab,
                                                          nullptr, status_word);
    WAR_LAUNCH_CHECK();
    // ---- host bookkeeping as of this point of the stream (undone below if anything fails to enqueue) ----
    try {
        for (int t = 1; t <= T; ++t) ix->bounds.push_back(M_old + (h_offsets[t] - h_offsets[0]) + t);
    } catch (...) {
        ix->bounds.resize((size_t)T_old + 1);
        return WAR_ERR_OOM;
    }
    ix->M = M;
    ix->T = T_old + T;
    const war_index_arrays old = ix->published();
    war_index_arrays& sh = ix->shadow();
    auto enqueue = [&]() -> war_status_t {
        if (merge) {
            const war_status_t st = sort_suffixes_full(ix->corpus + M_old, m, ix->T, ix->vocab, ix->max_depth, new_sa, sort_scratch, s);
            if (st != WAR_OK) return st;
            insert_pos_kernel<<<grid_for(m), kThreads, 0, s>>>(ix->corpus, old.sa, old.bucket, new_sa, m, M_old, ix->vocab, ix->max_depth, pos);
            WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(scan_temp, b_scan, pos, pos, MaxOp(), (int)m, s));
            WAR_CUDA_TRY(cudaMemsetAsync(add, 0, b_add, s));
            count_pos_kernel<<<grid_for(m), kThreads, 0, s>>>(pos, m, add);
            WAR_CUDA_TRY(cub::DeviceScan::InclusiveScan(scan_temp, b_scan, add, add, SumOp(), (int)(M_old + 1), s));
            scatter_old_kernel<<<grid_for(M_old), kThreads, 0, s>>>(old.sa, add, M_old, sh.sa);
            scatter_new_kernel<<<grid_for(m), kThreads, 0, s>>>(new_sa, pos, m, M_old, sh.sa);
        } else {
            const war_status_t st = sort_suffixes_full(ix->corpus, M, ix->T, ix->vocab, ix->max_depth, sh.sa, sort_scratch, s);
            if (st != WAR_OK) return st;
        }
        lcp_kernel<<<grid_for(M), kThreads, 0, s>>>(ix->corpus, sh.sa, M, ix->max_depth, sh.lcp);
        bucket_from_sa_kernel<<<grid_for(M + 1), kThreads, 0, s>>>(ix->corpus, sh.sa, M, ix->vocab, sh.bucket);
        WAR_LAUNCH_CHECK();
        WAR_CUDA_TRY(cudaMemsetAsync(sh.memo, 0, sizeof(int32_t) * kMemoEntries * kMemoInts, s));
        set_u32_kernel<<<1, 1, 0, s>>>(&ix->d_view->cur, (unsigned int)(ix->cur ^ 1));
        WAR_LAUNCH_CHECK();
        return WAR_OK;
    };
    const war_status_t st = enqueue();
    if (st != WAR_OK) {                                      // nothing was published: forget the addition
        ix->M = M_old;
        ix->T = T_old;
        ix->bounds.resize((size_t)T_old + 1);
        return st;
    }
    { std::lock_guard<std::mutex> g(ix->lock); ix->cur ^= 1; }
    return WAR_OK;
}

}  // namespace

extern "C" war_status_t war_index_append_async(war_index_t* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T,
                                               war_stream_t stream) {
    if (!ix) return WAR_ERR_INVALID_ARG;
    const war_status_t st = check_offsets(h_offsets, T);
    if (st != WAR_OK) return st;
    if (T == 0) return WAR_OK;
    return append_async(ix, d_tokens, h_offsets, T, stream);
}

extern "C" war_status_t war_index_build(const int32_t* d_tokens, const int64_t* h_offsets, int32_t T, int32_t vocab,
                                        int32_t max_depth, int64_t capacity_tokens, war_stream_t stream,
                                        war_index_t** out) {
    if (!out) return WAR_ERR_INVALID_ARG;
    *out = nullptr;
    if (vocab < 1 || max_depth < 1 || max_depth > 128 || capacity_tokens < 0) return WAR_ERR_INVALID_ARG;
    war_status_t st = check_offsets(h_offsets, T);
    if (st != WAR_OK) return st;
    if (capacity_tokens >= ((int64_t)1 << 31) - 256) return WAR_ERR_CAPACITY;
    war_index* ix = new (std::nothrow) war_index();
    if (!ix) return WAR_ERR_OOM;
    ix->vocab = vocab;
    ix->max_depth = max_depth;
    ix->capacity = capacity_tokens;
    cudaGetDevice(&ix->device);
    const int64_t cap = capacity_tokens > 0 ? capacity_tokens : 1;
    cudaError_t e = cudaMalloc((void**)&ix->corpus, sizeof(int32_t) * (cap + 128));   // +128: readable slack behind the last separator
    for (int k = 0; k < 2; ++k) {
        if (e == cudaSuccess) e = cudaMalloc((void**)&ix->set[k].sa, sizeof(int32_t) * cap);
        if (e == cudaSuccess) e = cudaMalloc((void**)&ix->set[k].lcp, cap + 64);
        if (e == cudaSuccess) e = cudaMalloc((void**)&ix->set[k].bucket, sizeof(int32_t) * (vocab + 1));
        if (e == cudaSuccess) e = cudaMalloc((void**)&ix->set[k].memo, sizeof(int32_t) * kMemoEntries * kMemoInts);
        if (e == cudaSuccess) e = cudaMemsetAsync(ix->set[k].memo, 0, sizeof(int32_t) * kMemoEntries * kMemoInts, stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(ix->set[k].lcp, 0, cap + 64, stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(ix->set[k].bucket, 0, sizeof(int32_t) * (vocab + 1), stream);
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(ix->corpus, 0xff, sizeof(int32_t) * (cap + 128), stream);
    if (e == cudaSuccess) e = cudaMalloc((void**)&ix->d_view, sizeof(war_index_view));
    if (e == cudaSuccess) e = cudaMallocHost((void**)&ix->h_stage, sizeof(int64_t) * war_index::kStageEntries);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ix->stage_free, cudaEventDisableTiming);
    if (e == cudaSuccess) {
        war_index_view v;
        v.set[0] = ix->set[0]; v.set[1] = ix->set[1]; v.cur = (unsigned int)ix->cur;
        e = cudaMemcpyAsync(ix->d_view, &v, sizeof(v), cudaMemcpyHostToDevice, stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(stream);            // (v is a local)
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        war_index_destroy(ix);
        return e == cudaErrorMemoryAllocation ? WAR_ERR_OOM : WAR_ERR_CUDA;
    }
    st = add_trajectories(ix, d_tokens, h_offsets, T, stream);
    if (st == WAR_OK) st = rebuild(ix, stream);
    if (st != WAR_OK) { war_index_destroy(ix); return st; }
    *out = ix;
    return WAR_OK;
}

extern "C" war_status_t war_index_append(war_index_t* ix, const int32_t* d_tokens, const int64_t* h_offsets, int32_t T,
                                         war_stream_t stream) {
    if (!ix) return WAR_ERR_INVALID_ARG;
    war_status_t st = check_offsets(h_offsets, T);
    if (st != WAR_OK) return st;
    if (T == 0) return WAR_OK;
    const int64_t M_old = ix->M;
    const int32_t T_old = ix->T;
    st = add_trajectories(ix, d_tokens, h_offsets, T, stream);
    if (st != WAR_OK) return st;
    // merging pays when the addition is the smaller part; otherwise sort everything again
    st = (M_old > 0 && ix->M - M_old < M_old) ? merge_new_suffixes(ix, M_old, stream) : rebuild(ix, stream);
    if (st != WAR_OK) {                                      // nothing was published: forget the addition
        ix->M = M_old;
        ix->T = T_old;
        ix->bounds.resize((size_t)T_old + 1);
    }
    return st;
}

extern "C" war_status_t war_index_evict(war_index_t* ix, int32_t n_oldest, war_stream_t stream) {
    if (!ix || n_oldest < 0 || n_oldest > ix->T) return WAR_ERR_INVALID_ARG;
    if (n_oldest == 0) return WAR_OK;
    return evict_oldest(ix, n_oldest, stream);
}

// ---- export / import ------------------------------------------------------------------------------
// Layout of an exported index (host memory, little endian): header, int64 bounds[T+1], int32 corpus[M], int32 sa[M],
// uint8 lcp[M] padded to 8 bytes, int32 bucket[vocab+1].
struct ExportHeader {
    uint64_t magic;              // "WARINDX1"
    int64_t M;
    int32_t T, vocab, max_depth, reserved;
};
constexpr uint64_t kExportMagic = 0x3158444e49524157ull;
static size_t pad8(size_t x) { return (x + 7) & ~(size_t)7; }
static size_t export_bytes(int64_t M, int32_t T, int32_t vocab) {
    return sizeof(ExportHeader) + sizeof(int64_t) * ((size_t)T + 1) + 2 * pad8(sizeof(int32_t) * (size_t)M) + pad8((size_t)M) +
           pad8(sizeof(int32_t) * ((size_t)vocab + 1));
}

extern "C" size_t war_index_export_bytes(const war_index_t* ix) {
    return ix ? export_bytes(ix->M, ix->T, ix->vocab) : 0;
}

extern "C" war_status_t war_index_export(const war_index_t* cix, void* h_dst, size_t bytes, war_stream_t stream) {
    war_index* ix = const_cast<war_index*>(cix);
    if (!ix || !h_dst || bytes < export_bytes(ix->M, ix->T, ix->vocab)) return WAR_ERR_INVALID_ARG;
    const war_index_arrays a = ix->published();
    const size_t M = (size_t)ix->M;
    char* at = (char*)h_dst;
    ExportHeader h = {kExportMagic, ix->M, ix->T, ix->vocab, ix->max_depth, 0};
    memcpy(at, &h, sizeof(h)); at += sizeof(h);
    memcpy(at, ix->bounds.data(), sizeof(int64_t) * ((size_t)ix->T + 1)); at += sizeof(int64_t) * ((size_t)ix->T + 1);
    WAR_CUDA_TRY(cudaMemcpyAsync(at, ix->corpus, sizeof(int32_t) * M, cudaMemcpyDeviceToHost, stream)); at += pad8(sizeof(int32_t) * M);
    WAR_CUDA_TRY(cudaMemcpyAsync(at, a.sa, sizeof(int32_t) * M, cudaMemcpyDeviceToHost, stream)); at += pad8(sizeof(int32_t) * M);
    WAR_CUDA_TRY(cudaMemcpyAsync(at, a.lcp, M, cudaMemcpyDeviceToHost, stream)); at += pad8(M);
    WAR_CUDA_TRY(cudaMemcpyAsync(at, a.bucket, sizeof(int32_t) * ((size_t)ix->vocab + 1), cudaMemcpyDeviceToHost, stream));
    WAR_CUDA_TRY(cudaStreamSynchronize(stream));
    // the few bytes that pad a section to 8 are defined too (an export is a function of the index alone)
    char* sec = (char*)h_dst + sizeof(ExportHeader) + sizeof(int64_t) * ((size_t)ix->T + 1);
    const size_t lens[4] = {sizeof(int32_t) * M, sizeof(int32_t) * M, M, sizeof(int32_t) * ((size_t)ix->vocab + 1)};
    for (int k = 0; k < 4; ++k) {
        memset(sec + lens[k], 0, pad8(lens[k]) - lens[k]);
        sec += pad8(lens[k]);
    }
    return WAR_OK;
}

extern "C" war_status_t war_index_import(const void* h_src, size_t bytes, int64_t capacity_tokens, war_stream_t stream,
                                         war_index_t** out) {
    if (!out) return WAR_ERR_INVALID_ARG;
    *out = nullptr;
    if (!h_src || bytes < sizeof(ExportHeader)) return WAR_ERR_INVALID_ARG;
    ExportHeader h;
    memcpy(&h, h_src, sizeof(h));
    if (h.magic != kExportMagic || h.M < 0 || h.T < 0 || h.vocab < 1 || h.max_depth < 1 || h.max_depth > 128 || h.M < h.T)
        return WAR_ERR_INVALID_ARG;
    if (bytes < export_bytes(h.M, h.T, h.vocab)) return WAR_ERR_INVALID_ARG;
    if (capacity_tokens < h.M) return WAR_ERR_CAPACITY;
    const char* at = (const char*)h_src + sizeof(h);
    const int64_t* bounds = (const int64_t*)at;
    if (bounds[0] != 0 || bounds[h.T] != h.M) return WAR_ERR_INVALID_ARG;
    for (int t = 0; t < h.T; ++t)
        if (bounds[t + 1] <= bounds[t]) return WAR_ERR_INVALID_ARG;     // every trajectory holds at least its separator
    // an empty index of that capacity, then the arrays
    const int64_t zero = 0;
    war_index_t* ix = nullptr;
    war_status_t st = war_index_build(nullptr, &zero, 0, h.vocab, h.max_depth, capacity_tokens, stream, &ix);
    if (st != WAR_OK) return st;
    const size_t M = (size_t)h.M;
    at += sizeof(int64_t) * ((size_t)h.T + 1);
    war_index_arrays& a = ix->shadow();
    cudaError_t e = cudaMemcpyAsync(ix->corpus, at, sizeof(int32_t) * M, cudaMemcpyHostToDevice, stream); at += pad8(sizeof(int32_t) * M);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.sa, at, sizeof(int32_t) * M, cudaMemcpyHostToDevice, stream);
    at += pad8(sizeof(int32_t) * M);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.lcp, at, M, cudaMemcpyHostToDevice, stream);
    at += pad8(M);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.bucket, at, sizeof(int32_t) * ((size_t)h.vocab + 1), cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(a.memo, 0, sizeof(int32_t) * kMemoEntries * kMemoInts, stream);
    if (e != cudaSuccess) { (void)cudaGetLastError(); war_index_destroy(ix); return WAR_ERR_CUDA; }
    try { ix->bounds.assign(bounds, bounds + h.T + 1); } catch (...) { war_index_destroy(ix); return WAR_ERR_OOM; }
    ix->M = h.M;
    ix->T = h.T;
    if (ix->publish(stream) != cudaSuccess) { (void)cudaGetLastError(); war_index_destroy(ix); return WAR_ERR_CUDA; }
    *out = ix;
    return WAR_OK;
}

extern "C" war_status_t war_index_info(const war_index_t* ix, war_index_info_t* out) {
    if (!ix || !out) return WAR_ERR_INVALID_ARG;
    out->M = ix->M;
    out->capacity_tokens = ix->capacity;
    out->T = ix->T;
    out->vocab = ix->vocab;
    out->max_depth = ix->max_depth;
    out->reserved = 0;
    const war_index_arrays a = const_cast<war_index*>(ix)->published();
    out->d_corpus = ix->corpus;
    out->d_sa = a.sa;
    out->d_lcp = a.lcp;
    out->d_bucket = a.bucket;
    return WAR_OK;
}

extern "C" war_status_t war_index_destroy(war_index_t* ix) {
    if (!ix) return WAR_OK;
    if (ix->corpus) cudaFree(ix->corpus);
    if (ix->d_view) cudaFree(ix->d_view);
    if (ix->h_stage) cudaFreeHost(ix->h_stage);
    if (ix->stage_free) cudaEventDestroy(ix->stage_free);
    for (int k = 0; k < 2; ++k) {
        if (ix->set[k].sa) cudaFree(ix->set[k].sa);
        if (ix->set[k].lcp) cudaFree(ix->set[k].lcp);
        if (ix->set[k].bucket) cudaFree(ix->set[k].bucket);
        if (ix->set[k].memo) cudaFree(ix->set[k].memo);
    }
    delete ix;
    return WAR_OK;
}
