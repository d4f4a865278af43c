// Accept: longest root path of the draft tree that equals the target model's own tokens.
// One warp per request.  Slots are stored parent-before-child, so one in-order sweep settles every slot.
#include "war_common.cuh"

namespace {

constexpr int kMaxSlots = 64;

__global__ void war_accept_kernel(const int32_t* __restrict__ ids, const int32_t* __restrict__ parent,
                                  const int32_t* __restrict__ num_nodes, const int32_t* __restrict__ target,
                                  int B, int N, int mode,
                                  int32_t* __restrict__ accept_len, int32_t* __restrict__ accept_path,
                                  int32_t* __restrict__ bonus, int* status_word) {
    const int warps_per_block = blockDim.x / 32;
    const int b = blockIdx.x * warps_per_block + threadIdx.x / 32;
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    __shared__ int s_parent[4][kMaxSlots];
    __shared__ int s_depth[4][kMaxSlots];        // -1 = some slot on the root path does not match
    __shared__ int s_target[4][kMaxSlots];
    int* par = s_parent[threadIdx.x / 32];
    int* dep = s_depth[threadIdx.x / 32];
    int* tgt = s_target[threadIdx.x / 32];

    // The whole rows are requested at once, whatever num_nodes says (rows are N long; entries at or beyond num_nodes
    // are read and ignored): one memory latency instead of the chain num_nodes -> parent -> target[parent].
    int n = num_nodes[b];
    int p_in[2], id_in[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = lane + 32 * h;
        p_in[h] = -1; id_in[h] = 0;
        if (j < N) {
            p_in[h] = parent[(size_t)b * N + j];
            id_in[h] = ids[(size_t)b * N + j];
            tgt[j] = target[(size_t)b * N + j];
        }
    }
    bool bad = n < 0 || n > N;
    if (bad) n = 0;
    __syncwarp();
    // matched[j] per lane-owned slot; parents validated here
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int j = lane + 32 * h;
        if (j >= N) continue;
        int p = -1, m = 0;
        if (j < n) {
            p = p_in[h];
            if (j == 0) {
                m = 1;
            } else if (p < 0 || p >= j) {
                bad = true;
            } else {
                const int want = mode == 0 ? tgt[p] : tgt[j];
                m = id_in[h] == want;
            }
        }
        par[j] = p;
        dep[j] = m;                               // holds matched[j] until the sweep below
    }
    bad = __any_sync(0xffffffffu, bad);
    __syncwarp();
    if (bad) {
        if (lane == 0) { war_set_device_status(status_word, WAR_ERR_BAD_TREE); accept_len[b] = 0; bonus[b] = -1; }
        for (int j = lane; j < N; j += 32) accept_path[(size_t)b * N + j] = -1;
        return;
    }
    int best_slot = 0, best_depth = 0;
    if (lane == 0) {
        // ok(j) = matched(j) && ok(parent); depth from the same pass.  Strict '>' keeps the lowest slot on ties.
        for (int j = 0; j < n; ++j) {
            int d;
            if (j == 0) d = 0;
            else d = (dep[j] && dep[par[j]] >= 0) ? dep[par[j]] + 1 : -1;
            dep[j] = d;
            if (d > best_depth) { best_depth = d; best_slot = j; }
        }
    }
    best_slot = __shfl_sync(0xffffffffu, best_slot, 0);
    best_depth = __shfl_sync(0xffffffffu, best_depth, 0);
    __syncwarp();
    for (int j = lane; j < N; j += 32)
        if (j >= best_depth) accept_path[(size_t)b * N + j] = -1;
    if (lane == 0) {
        int a = best_slot;
        for (int d = best_depth - 1; d >= 0; --d) { accept_path[(size_t)b * N + d] = a; a = par[a]; }
        accept_len[b] = best_depth;
        bonus[b] = (mode == 0 && n > 0) ? tgt[best_slot] : -1;
    }
}

}  // namespace

extern "C" war_status_t war_accept(const int32_t* d_ids, const int32_t* d_parent, const int32_t* d_num_nodes,
                                   const int32_t* d_target_ids, int32_t B, int32_t N, int32_t target_mode,
                                   int32_t* d_accept_len, int32_t* d_accept_path, int32_t* d_bonus,
                                   war_stream_t stream) {
    if (B < 0 || N < 1 || N > kMaxSlots || (target_mode != 0 && target_mode != 1)) return WAR_ERR_INVALID_ARG;
    if (B == 0) return WAR_OK;
    if (!d_ids || !d_parent || !d_num_nodes || !d_target_ids || !d_accept_len || !d_accept_path || !d_bonus)
        return WAR_ERR_INVALID_ARG;
    int* status_word = war_status_word();
    if (!status_word) return WAR_ERR_CUDA;
    const int warps = 4;
    war_accept_kernel<<<(B + warps - 1) / warps, warps * 32, 0, stream>>>(
        d_ids, d_parent, d_num_nodes, d_target_ids, B, N, target_mode, d_accept_len, d_accept_path, d_bonus, status_word);
    WAR_LAUNCH_CHECK();
    return WAR_OK;
}
