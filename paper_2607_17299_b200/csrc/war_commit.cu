// Commit: the accepted path becomes the end of each request's context.
//   kv kernel   one CTA per (request, kv head): the K/V rows of the accepted slots move to the positions right after
//               the root.  Every row is read into registers before any row of that head is written, because a
//               destination may be another move's source (path [2, 4]: position +2 is read by the first move and
//               written by the second).
//   ctx kernel  one warp per request, after the kv kernel in stream order (it changes prefix_len, which the kv kernel
//               reads): tail window, tail length, prefix length.
// Both kernels check the path the same way and leave a malformed request untouched.
#include <cuda_bf16.h>
#include "war_common.cuh"

namespace {

constexpr int kMaxSlots = 64;
constexpr int kMaxTail = 32;
constexpr int kKvThreads = 256;
constexpr int kPiecesPerRow = 16;            // 128 bf16 = 16 pieces of 16 bytes
constexpr int kMaxPerThread = (kMaxSlots * 2 * kPiecesPerRow + kKvThreads - 1) / kKvThreads;

struct Strides { long long s[4]; };

// accept_len in [0, N), slots strictly increasing inside [1, N): a root path in slot order
__device__ __forceinline__ bool path_ok(const int32_t* __restrict__ path, int k, int N) {
    if (k < 0 || k >= N) return false;
    int prev = 0;
    for (int d = 0; d < k; ++d) {
        const int s = path[d];
        if (s <= prev || s >= N) return false;
        prev = s;
    }
    return true;
}

__global__ void __launch_bounds__(kKvThreads)
war_commit_kv_kernel(const int32_t* __restrict__ accept_len, const int32_t* __restrict__ accept_path,
                     const int32_t* __restrict__ page_table, const int32_t* __restrict__ prefix_len,
                     __nv_bfloat16* kpool, __nv_bfloat16* vpool, Strides ks, Strides vs, int N, int page_size, int max_pages,
                     long long num_pages, int* status_word) {
    const int b = blockIdx.x, h = blockIdx.y;
    __shared__ int s_path[kMaxSlots];
    __shared__ int s_ok;
    const int k = accept_len[b];
    const int pl = prefix_len[b];
    if (threadIdx.x == 0) {
        bool ok = pl >= 0 && path_ok(accept_path + (size_t)b * N, k, N);
        if (ok && k > 0) ok = (pl + accept_path[(size_t)b * N + k - 1]) / page_size < max_pages;
        s_ok = ok;
    }
    for (int d = threadIdx.x; d < N; d += kKvThreads) s_path[d] = accept_path[(size_t)b * N + d];
    __syncthreads();
    if (!s_ok || k == 0) return;
    const int32_t* pt = page_table + (size_t)b * max_pages;
    auto row_ptr = [&](int which, int pos) -> uint4* {
        long long page = pt[pos / page_size];
        if (page < 0 || page >= num_pages) { war_set_device_status(status_word, WAR_ERR_BAD_PAGE); return nullptr; }
        const Strides& st = which ? vs : ks;
        __nv_bfloat16* base = which ? vpool : kpool;
        return reinterpret_cast<uint4*>(base + page * st.s[0] + (long long)h * st.s[1] + (long long)(pos % page_size) * st.s[2]);
    };
    // item = (move d, K or V, 16-byte piece); a move whose row is already in place is skipped on both sides
    const int items = k * 2 * kPiecesPerRow;
    uint4 buf[kMaxPerThread];
    unsigned have = 0;                                           // bit r: buf[r] holds a row piece that was really read
#pragma unroll
    for (int r = 0; r < kMaxPerThread; ++r) {
        const int it = threadIdx.x + r * kKvThreads;
        buf[r] = make_uint4(0, 0, 0, 0);
        if (it < items) {
            const int d = it / (2 * kPiecesPerRow), which = (it / kPiecesPerRow) & 1, piece = it % kPiecesPerRow;
            if (s_path[d] != d + 1) {
                const uint4* src = row_ptr(which, pl + s_path[d]);
                if (src) { buf[r] = src[piece]; have |= 1u << r; }
            }
        }
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < kMaxPerThread; ++r) {
        const int it = threadIdx.x + r * kKvThreads;
        if (it < items) {
            const int d = it / (2 * kPiecesPerRow), which = (it / kPiecesPerRow) & 1, piece = it % kPiecesPerRow;
            if (s_path[d] != d + 1 && ((have >> r) & 1u)) {        // a row whose source page was bad is skipped, not zeroed
                uint4* dst = row_ptr(which, pl + 1 + d);
                if (dst) dst[piece] = buf[r];
            }
        }
    }
}

__global__ void war_commit_ctx_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ accept_len,
                                      const int32_t* __restrict__ accept_path, const int32_t* __restrict__ bonus,
                                      int B, int N, int P, int page_size, int max_pages, int32_t* prefix_len,
                                      int32_t* tail, int32_t* tail_len, int* status_word) {
    const int b = blockIdx.x * (blockDim.x / 32) + threadIdx.x / 32;
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    const int k = accept_len[b], pl = prefix_len[b], tl = tail_len[b], bn = bonus[b];
    if (tl < 0) return;                                                    // not running (see war_draft): nothing to advance
    bool ok = pl >= 0 && tl >= 0 && tl <= P && path_ok(accept_path + (size_t)b * N, k, N);
    if (ok && k > 0) ok = (pl + accept_path[(size_t)b * N + k - 1]) / page_size < max_pages;
    if (!ok) {
        if (lane == 0) war_set_device_status(status_word, WAR_ERR_BAD_TREE);
        return;
    }
    // context' = old window ++ accepted ids ++ bonus (if any); the new window is its last min(P, length) tokens
    const int added = k + (bn >= 0 ? 1 : 0);
    const int total = tl + added;
    const int new_len = total < P ? total : P;
    int v = 0;
    if (lane < P && lane >= P - new_len) {
        const int idx = total - new_len + (lane - (P - new_len));          // index into context'
        if (idx < tl) v = tail[(size_t)b * P + (P - tl + idx)];
        else {
            const int y = idx - tl;
            v = y < k ? ids[(size_t)b * N + accept_path[(size_t)b * N + y]] : bn;
        }
    }
    __syncwarp();                                                          // every read of the old window is done
    if (lane < P) tail[(size_t)b * P + lane] = v;
    if (lane == 0) {
        tail_len[b] = new_len;
        prefix_len[b] = pl + added;
    }
}

}  // namespace

extern "C" war_status_t war_commit(const int32_t* d_ids, const int32_t* d_accept_len, const int32_t* d_accept_path,
                                   const int32_t* d_bonus, void* d_kpool, void* d_vpool, const int32_t* d_page_table,
                                   const war_commit_params_t* p, int32_t* d_prefix_len, int32_t* d_tail,
                                   int32_t* d_tail_len, war_stream_t stream) {
    if (!p) return WAR_ERR_INVALID_ARG;
    if (p->B < 0 || p->N < 1 || p->N > kMaxSlots || p->P < 1 || p->P > kMaxTail || p->Hkv < 1 || p->page_size < 1 ||
        p->max_pages_per_req < 1 || p->num_pages < 1)
        return WAR_ERR_INVALID_ARG;
    if (p->D != 128) return WAR_ERR_UNSUPPORTED;
    if (p->B == 0) return WAR_OK;
    if (!d_ids || !d_accept_len || !d_accept_path || !d_bonus || !d_kpool || !d_vpool || !d_page_table || !d_prefix_len ||
        !d_tail || !d_tail_len)
        return WAR_ERR_INVALID_ARG;
    // rows are moved 16 bytes at a time: unit stride along d, every other stride and both bases 16-byte aligned
    Strides ks, vs;
    for (int i = 0; i < 4; ++i) { ks.s[i] = p->k_strides[i]; vs.s[i] = p->v_strides[i]; }
    if (ks.s[3] != 1 || vs.s[3] != 1) return WAR_ERR_UNSUPPORTED;
    for (int i = 0; i < 3; ++i)
        if (ks.s[i] < 0 || vs.s[i] < 0 || (ks.s[i] & 7) || (vs.s[i] & 7)) return WAR_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(d_kpool) & 15) || (reinterpret_cast<uintptr_t>(d_vpool) & 15)) return WAR_ERR_UNSUPPORTED;
    if (p->Hkv > 65535) return WAR_ERR_UNSUPPORTED;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    war_commit_kv_kernel<<<dim3(p->B, p->Hkv), kKvThreads, 0, stream>>>(
        d_accept_len, d_accept_path, d_page_table, d_prefix_len, (__nv_bfloat16*)d_kpool, (__nv_bfloat16*)d_vpool, ks, vs, p->N,
        p->page_size, p->max_pages_per_req, p->num_pages, status_word);
    WAR_LAUNCH_CHECK();
    const int warps = 4;
    war_commit_ctx_kernel<<<(p->B + warps - 1) / warps, warps * 32, 0, stream>>>(
        d_ids, d_accept_len, d_accept_path, d_bonus, p->B, p->N, p->P, p->page_size, p->max_pages_per_req, d_prefix_len,
        d_tail, d_tail_len, status_word);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
