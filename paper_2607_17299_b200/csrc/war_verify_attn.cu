// Verify attention: argument checks, the planning kernel, the split-KV combine kernel and the plain CUDA-core
// attention kernel (kept as the A/B reference of the tensor-core kernel in war_verify_attn_sm100.cu).
#include <cuda_bf16.h>
#include <math_constants.h>
#include "war_common.cuh"
#include "war_attn_plan.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ------------------------------------------------------------------------------------------------
// plan: one CTA
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
attn_plan_kernel(const int32_t* __restrict__ prefix_len, const int32_t* __restrict__ num_nodes,
                 const int32_t* __restrict__ parent, int B, int N, int Hkv, int G, int page_size, int max_pages,
                 AttnWorkspace w, int* status_word) {
    constexpr int kPer = kMaxPlanB / 1024;    // requests per thread, kept in registers through all phases
    __shared__ int s_tiles[kMaxPlanB];
    __shared__ int s_units[kMaxPlanB];        // units per request, indexed by sorted position; then exclusive scan
    __shared__ int s_red[32];
    __shared__ long long s_sum[32];
    __shared__ int s_chunk_tiles;
    const int tid = threadIdx.x;
    int r_n[kPer], r_tiles[kPer], r_rbs[kPer], r_pos[kPer], r_nc[kPer];
    // per request: validate, ancestor masks, tile count
    long long my_tiles = 0;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int i = tid + k * 1024;
        r_n[k] = 0; r_tiles[k] = 0; r_rbs[k] = 0; r_pos[k] = 0; r_nc[k] = 0;
        if (i >= B) continue;
        int n = num_nodes[i];
        const int pl = prefix_len[i];
        bool bad = n < 0 || n > N || pl < 0;
        if (!bad && n > 0) {
            // all parent ids of the request are requested before any is used, so their latencies overlap
            int pbuf[64];
            const int4* prow = reinterpret_cast<const int4*>(parent + (size_t)i * N);
            if ((N & 3) == 0 && (reinterpret_cast<uintptr_t>(parent) & 15) == 0) {
                for (int j = 0; j < n; j += 4) {
                    const int4 v = prow[j >> 2];
                    pbuf[j] = v.x; pbuf[j + 1] = v.y; pbuf[j + 2] = v.z; pbuf[j + 3] = v.w;
                }
            } else {
                for (int j = 0; j < n; ++j) pbuf[j] = parent[(size_t)i * N + j];
            }
            uint64_t local[64];
            local[0] = 1ull;
            for (int j = 1; j < n; ++j) {
                const int p = pbuf[j];
                if (p < 0 || p >= j) { bad = true; break; }
                local[j] = local[p] | (1ull << j);
            }
            if (!bad)
                for (int j = 0; j < n; ++j) w.anc[(size_t)i * N + j] = local[j];
        }
        if (bad) { war_set_device_status(status_word, WAR_ERR_BAD_TREE); n = 0; }
        int tiles = 0;
        if (n > 0) {
            const long long L = (long long)pl + n;
            if ((L + page_size - 1) / page_size > max_pages) { war_set_device_status(status_word, WAR_ERR_BAD_PAGE); n = 0; }
            else tiles = (int)((L + kTileKeys - 1) / kTileKeys);
        }
        s_tiles[i] = tiles;
        r_n[k] = n; r_tiles[k] = tiles;
        r_rbs[k] = n > 0 ? (G * n + kRowBlock - 1) / kRowBlock : 0;
        my_tiles += (long long)tiles * r_rbs[k];
    }
    // block sum of tiles (weighted by row blocks and kv heads)
    for (int o = 16; o > 0; o >>= 1) my_tiles += __shfl_xor_sync(0xffffffffu, my_tiles, o);
    if ((tid & 31) == 0) s_sum[tid >> 5] = my_tiles;
    __syncthreads();
    if (tid == 0) {
        long long tot = 0;
        for (int i = 0; i < (int)(blockDim.x >> 5); ++i) tot += s_sum[i];
        tot *= Hkv;
        long long ct = (tot + kTargetUnits - 1) / kTargetUnits;
        if (ct < kMinChunkTiles) ct = kMinChunkTiles;
        s_chunk_tiles = (int)ct;
        w.counters[0] = 0;
        w.counters[2] = (int)ct;
    }
    __syncthreads();
    const int chunk_tiles = s_chunk_tiles;
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
        r_nc[k] = t > 0 ? (t + chunk_tiles - 1) / chunk_tiles : 0;
        s_units[pos] = r_nc[k] * Hkv * r_rbs[k];
    }
    __syncthreads();
    // exclusive scan of s_units: per-thread serial segments + warp scans
    {
        const int per = (B + blockDim.x - 1) / blockDim.x;
        const int b0 = tid * per, b1 = min(B, b0 + per);
        int sum = 0;
        for (int q = b0; q < b1; ++q) sum += s_units[q];
        int incl = sum;
        for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if ((tid & 31) >= o) incl += y; }
        if ((tid & 31) == 31) s_red[tid >> 5] = incl;
        __syncthreads();
        if (tid < 32) {
            int x = s_red[tid], xi = x;
            for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, xi, o); if (tid >= o) xi += y; }
            s_red[tid] = xi - x;
            if (tid == 31) w.counters[1] = xi;     // total number of units
        }
        __syncthreads();
        int run = s_red[tid >> 5] + incl - sum;
        for (int q = b0; q < b1; ++q) { const int u = s_units[q]; s_units[q] = run; run += u; }
    }
    __syncthreads();
    // unit table: per request, chunks balanced to within one tile, order (chunk, kv head, row block)
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
        const int i = tid + k * 1024;
        if (i >= B) continue;
        const int base = s_units[r_pos[k]];
        const int nc = r_nc[k], t = r_tiles[k], rbs = r_rbs[k];
        AttnReq rq;
        rq.base_unit = base; rq.n_chunks = nc; rq.n_tiles = t; rq.n_nodes = r_n[k];
        w.req[i] = rq;
        int u = base;
        for (int c = 0; c < nc; ++c) {
            const int tb = (int)((long long)t * c / nc), te = (int)((long long)t * (c + 1) / nc);
            for (int h = 0; h < Hkv; ++h)
                for (int rb = 0; rb < rbs; ++rb, ++u) {
                    AttnUnit x;
                    x.req = i; x.kvh = h; x.rb = rb; x.tile_begin = tb; x.tile_end = te; x.n_chunks = nc; x.chunk = c; x.pad = 0;
                    w.units[u] = x;
                }
        }
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
    const int u0 = rq.base_unit + kvh * rbs + rb, ustep = Hkv * rbs;       // unit of chunk c = u0 + c * ustep
    float M = -CUDART_INF_F;
    for (int c = lane; c < rq.n_chunks; c += 32)
        M = fmaxf(M, w.part_ml[((size_t)(u0 + c * ustep) * w.rows + rr) * 2]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
    float l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = 0; c < rq.n_chunks; ++c) {
        const size_t base = (size_t)(u0 + c * ustep) * w.rows + rr;
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
                   long long num_pages, float scale_log2, AttnWorkspace w, __nv_bfloat16* __restrict__ out,
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
                    const size_t off = (((size_t)page * Hkv + un.kvh) * page_size + pos % page_size) * 128 + piece * 8;
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

bool contiguous_head_major(const int64_t* s, const war_attn_params_t* p) {
    return s[3] == 1 && s[2] == p->D && s[1] == (int64_t)p->page_size * p->D &&
           s[0] == (int64_t)p->Hkv * p->page_size * p->D;
}

war_status_t check_params(const war_attn_params_t* p) {
    if (!p) return WAR_ERR_INVALID_ARG;
    if (p->B < 0 || p->N < 1 || p->N > 64 || p->Hq < 1 || p->Hkv < 1 || p->Hq % p->Hkv != 0 || p->max_pages_per_req < 0 ||
        p->num_pages < 0 || p->kernel < 0 || p->kernel > 1 || !(p->scale > 0.f))
        return WAR_ERR_INVALID_ARG;
    if (p->D != 128 || (p->page_size != 16 && p->page_size != 32)) return WAR_ERR_UNSUPPORTED;
    if ((p->Hq / p->Hkv) * p->N > 512 || p->B > kMaxPlanB) return WAR_ERR_UNSUPPORTED;
    if (!contiguous_head_major(p->k_strides, p) || !contiguous_head_major(p->v_strides, p)) return WAR_ERR_UNSUPPORTED;
    return WAR_OK;
}

}  // namespace

war_status_t war_attn_launch_simple(const void* q, const void* k, const void* v, const int32_t* page_table,
                                    const int32_t* prefix_len, const war_attn_params_t* p, const AttnWorkspace& w,
                                    void* out, float* lse, int* status_word, cudaStream_t s) {
    const int G = p->Hq / p->Hkv;
    attn_simple_kernel<<<148 * 4, 128, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, page_table,
                                              prefix_len, p->N, p->Hq, p->Hkv, G, p->page_size, p->max_pages_per_req,
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
    attn_plan_kernel<<<1, 1024, 0, stream>>>(d_prefix_len, d_num_nodes, d_parent, p->B, p->N, p->Hkv, G, p->page_size,
                                            p->max_pages_per_req, w, status_word);
    WAR_LAUNCH_CHECK();
    if (p->kernel == 1)
        st = war_attn_launch_simple(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, p, w, d_out, d_lse, status_word, stream);
    else
        st = war_attn_launch_sm100(d_q, d_kpool, d_vpool, d_page_table, d_prefix_len, p, w, d_out, d_lse, status_word, stream);
    if (st != WAR_OK) return st;
    attn_combine_kernel<<<dim3(p->B * p->Hkv, (G * p->N + kCombineWarps - 1) / kCombineWarps), kCombineWarps * 32, 0, stream>>>(
        w, p->N, p->Hq, p->Hkv, G, (__nv_bfloat16*)d_out, d_lse);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
