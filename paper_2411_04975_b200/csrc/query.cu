// Read-only queries on a store: COUNT of token paths (the quantity Eq. 1
// divides), per-slot and store-wide bookkeeping.
#include "common.cuh"

namespace {

__global__ void query_counts_kernel(sd_store sv, int n, const int32_t* d_tree, const int64_t* d_offsets,
                                    const int32_t* d_paths, int32_t* d_counts) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int tree = d_tree[i];
    const long long b = d_offsets[i], e = d_offsets[i + 1];
    const int len = (int)(e - b);
    int count = 0;
    if (tree >= -1 && tree < sv.R && len >= 1 && len <= sv.D) {
        const int4* ent = tree < 0 ? sv.g_ent : sv.s_ent + (long long)tree * sv.spn;
        const int32_t* root = tree < 0 ? sv.g_root : sv.s_root + (long long)tree * sv.V;
        int x = d_paths[b];
        int node = (x >= 0 && x < sv.V) ? root[x] : -1;
        for (int k = 1; k < len && node >= 0; ++k) {
            const int4 pe = ent[node];
            const int cb = pe.z, nc = (int)((unsigned)pe.w & RUN_COUNT_MASK);
            x = d_paths[b + k];
            int lo = 0, hi = nc;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (ent[cb + mid].x < x) lo = mid + 1; else hi = mid;
            }
            node = (lo < nc && ent[cb + lo].x == x) ? cb + lo : -1;
        }
        if (node >= 0) count = ent[node].y;
    }
    d_counts[i] = count;
}

__global__ void slot_info_kernel(sd_store sv, int n, const int32_t* d_slot, int32_t* d_len, int32_t* d_nodes,
                                 int32_t* d_status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int slot = d_slot[i];
    int len = 0, nodes = 0, status = SD_STATUS_BAD_SLOT;
    if (slot >= 0 && slot < sv.R) {
        const SlotState* ss = sv.s_state + slot;
        len = ss->len; nodes = ss->live; status = ss->status;
    }
    if (d_len) d_len[i] = len;
    if (d_nodes) d_nodes[i] = nodes;
    if (d_status) d_status[i] = status;
}

}  // namespace

extern "C" int sd_query_counts(sd_store* s, int32_t n, const int32_t* d_tree, const int64_t* d_offsets,
                               const int32_t* d_paths, int32_t* d_counts, void* stream) {
    if (!s || n < 0) return SD_ERR_INVALID_ARG;
    if (n == 0) return SD_OK;
    if (!d_tree || !d_offsets || !d_paths || !d_counts) return SD_ERR_INVALID_ARG;
    query_counts_kernel<<<(unsigned)((n + 127) / 128), 128, 0, (cudaStream_t)stream>>>(*s, n, d_tree, d_offsets, d_paths,
                                                                                     d_counts);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}

extern "C" int sd_slot_info(sd_store* s, int32_t n, const int32_t* d_slot, int32_t* d_len, int32_t* d_nodes,
                            int32_t* d_status, void* stream) {
    if (!s || n < 0) return SD_ERR_INVALID_ARG;
    if (n == 0) return SD_OK;
    if (!d_slot) return SD_ERR_INVALID_ARG;
    slot_info_kernel<<<(unsigned)((n + 127) / 128), 128, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_len, d_nodes,
                                                                                  d_status);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}

extern "C" int sd_stats(sd_store* s, sd_stats_t* out, void* stream) {
    if (!s || !out) return SD_ERR_INVALID_ARG;
    GlobalState g;
    SD_CUDA_OK(cudaMemcpyAsync(&g, s->g_state, sizeof(g), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    SD_CUDA_OK(cudaStreamSynchronize((cudaStream_t)stream));
    out->global_nodes = g.live;
    out->global_pool_used = g.used;
    out->global_pool_cap = s->g_cap;
    out->global_tokens = g.tokens;
    out->slot_pool_nodes = s->spn;
    out->device_bytes = s->device_bytes;
    out->global_status = g.status;
    return SD_OK;
}
