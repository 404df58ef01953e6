// Read-only queries on a store: COUNT of token paths (the quantity Eq. 1
// divides), every node of a tree as a record, empirical entropy, per-slot and store-wide bookkeeping.
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
    SD_CHECK_DEVICE(s);
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
    SD_CHECK_DEVICE(s);
    if (n == 0) return SD_OK;
    if (!d_slot) return SD_ERR_INVALID_ARG;
    slot_info_kernel<<<(unsigned)((n + 127) / 128), 128, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_len, d_nodes,
                                                                                  d_status);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}

extern "C" int sd_stats(sd_store* s, sd_stats_t* out, void* stream) {
    if (!s || !out) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
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

// ---------------------------------------------------------------------------------------------
// Empirical entropy of a tree (Appendix "Predicting SuffixDecoding Effectiveness"): for every
// node the entropy of its children's count distribution, averaged over the nodes with the
// sibling sum as weight.  Level-by-level traversal from the root table (the pools also hold
// abandoned runs and top-block copies, so a plain sweep over the pool would count too much).
namespace {

__device__ __forceinline__ void warp_accumulate(double h_times_s, unsigned long long s, double* acc,
                                                unsigned long long* wsum) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        h_times_s += __shfl_xor_sync(0xffffffffu, h_times_s, o);
        s += __shfl_xor_sync(0xffffffffu, s, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (h_times_s != 0.0) atomicAdd(acc, h_times_s);
        if (s) atomicAdd(wsum, s);
    }
}

// depth-1 nodes: total count, and the first frontier
__global__ void entropy_root_sum_kernel(const int4* ent, const int32_t* root, int V, unsigned long long* total,
                                        int* frontier, int* n_frontier) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long c = 0;
    if (v < V) {
        const int idx = root[v];
        if (idx >= 0) {
            const int4 e = ent[idx];
            c = (unsigned)e.y;
            if ((unsigned)e.w & RUN_COUNT_MASK) frontier[atomicAdd(n_frontier, 1)] = idx;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((threadIdx.x & 31) == 0 && c) atomicAdd(total, c);
}

__global__ void entropy_root_kernel(const int4* ent, const int32_t* root, int V, const unsigned long long* total,
                                    double* acc, unsigned long long* wsum) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    double part = 0.0;                                           // -(c/S) log2(c/S) * S = -c log2(c/S)
    const double S = (double)*total;
    if (v < V) {
        const int idx = root[v];
        if (idx >= 0) { const double c = (double)(unsigned)ent[idx].y; part = -c * log2(c / S); }
    }
    warp_accumulate(part, 0ull, acc, wsum);
    if (blockIdx.x == 0 && threadIdx.x == 0 && *total) atomicAdd(wsum, *total);
}

// one thread per node of the current level
__global__ void entropy_level_kernel(const int4* ent, const int* frontier, int n, int* next, int* n_next, double* acc,
                                     unsigned long long* wsum) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    double part = 0.0;
    unsigned long long S = 0;
    if (i < n) {
        const int4 e = ent[frontier[i]];
        const int cb = e.z, nc = (int)((unsigned)e.w & RUN_COUNT_MASK);
        for (int k = 0; k < nc; ++k) S += (unsigned)ent[cb + k].y;
        const double dS = (double)S;
        for (int k = 0; k < nc; ++k) {
            const int4 c = ent[cb + k];
            const double dc = (double)(unsigned)c.y;
            part -= dc * log2(dc / dS);
            if ((unsigned)c.w & RUN_COUNT_MASK) next[atomicAdd(n_next, 1)] = cb + k;
        }
    }
    warp_accumulate(part, S, acc, wsum);
}

}  // namespace

extern "C" int sd_entropy(sd_store* s, int32_t tree, double* h_entropy, void* stream) {
    if (!s || !h_entropy || tree < -1 || tree >= s->R) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    cudaStream_t st = (cudaStream_t)stream;
    const int4* ent = tree < 0 ? s->g_ent : s->s_ent + (long long)tree * s->spn;
    const int32_t* root = tree < 0 ? s->g_root : s->s_root + (long long)tree * s->V;
    int live = 0;
    if (tree < 0) {
        GlobalState g;
        SD_CUDA_OK(cudaMemcpyAsync(&g, s->g_state, sizeof(g), cudaMemcpyDeviceToHost, st));
        SD_CUDA_OK(cudaStreamSynchronize(st));
        live = g.live;
    } else {
        SlotState ss;
        SD_CUDA_OK(cudaMemcpyAsync(&ss, s->s_state + tree, sizeof(ss), cudaMemcpyDeviceToHost, st));
        SD_CUDA_OK(cudaStreamSynchronize(st));
        live = ss.live;
    }
    *h_entropy = 0.0;
    if (live <= 0) return SD_OK;
    int *fa = nullptr, *fb = nullptr;
    unsigned char* small = nullptr;                              // total, acc, wsum, counters
    if (cudaMalloc(&fa, sizeof(int) * (size_t)live) != cudaSuccess || cudaMalloc(&fb, sizeof(int) * (size_t)live) != cudaSuccess ||
        cudaMalloc(&small, 64) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(fa); cudaFree(fb); cudaFree(small);
        return SD_ERR_NOMEM;
    }
    unsigned long long* total = (unsigned long long*)small;
    double* acc = (double*)(small + 8);
    unsigned long long* wsum = (unsigned long long*)(small + 16);
    int* cnt = (int*)(small + 24);                               // cnt[0], cnt[1]: frontier sizes
    cudaError_t ce = cudaMemsetAsync(small, 0, 64, st);
    entropy_root_sum_kernel<<<(s->V + 255) / 256, 256, 0, st>>>(ent, root, s->V, total, fa, cnt);
    entropy_root_kernel<<<(s->V + 255) / 256, 256, 0, st>>>(ent, root, s->V, total, acc, wsum);
    int n = 0, cur = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&n, cnt, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    for (int depth = 1; ce == cudaSuccess && n > 0 && depth <= SD_MAX_DEPTH; ++depth) {
        int* from = cur ? fb : fa;
        int* to = cur ? fa : fb;
        ce = cudaMemsetAsync(cnt + (cur ^ 1), 0, sizeof(int), st);
        entropy_level_kernel<<<(n + 255) / 256, 256, 0, st>>>(ent, from, n, to, cnt + (cur ^ 1), acc, wsum);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync(&n, cnt + (cur ^ 1), sizeof(int), cudaMemcpyDeviceToHost, st);
        if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
        cur ^= 1;
    }
    double h_acc = 0.0;
    unsigned long long h_w = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_acc, acc, sizeof(double), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_w, wsum, sizeof(h_w), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    cudaFree(fa); cudaFree(fb); cudaFree(small);
    if (ce != cudaSuccess) return SD_ERR_CUDA;
    *h_entropy = h_w ? h_acc / (double)h_w : 0.0;
    return SD_OK;
}

// ---------------------------------------------------------------------------------------------
// sd_enumerate: every node of a tree, level by level (a node's record comes after its parent's).
namespace {

// depth 1: the nodes the root table points at
__global__ void enumerate_root_kernel(const int4* ent, const int32_t* root, int V, long long max_nodes, int32_t* parent,
                                      int32_t* token, int32_t* count, int32_t* depth, int* next_ent, int* next_rec,
                                      int* n_next, unsigned long long* n_out) {
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= V || root[v] < 0) return;
    const int4 e = ent[root[v]];
    const unsigned long long o = atomicAdd(n_out, 1ull);
    if ((long long)o < max_nodes) { parent[o] = -1; token[o] = e.x; count[o] = e.y; depth[o] = 1; }
    if (((unsigned)e.w & RUN_COUNT_MASK) && (long long)o < max_nodes) {
        const int q = atomicAdd(n_next, 1);
        next_ent[q] = root[v]; next_rec[q] = (int)o;
    }
}

// one thread per node of the current level: a record for each of its children
__global__ void enumerate_level_kernel(const int4* ent, const int* cur_ent, const int* cur_rec, int n, int level,
                                       long long max_nodes, int32_t* parent, int32_t* token, int32_t* count, int32_t* depth,
                                       int* next_ent, int* next_rec, int* n_next, unsigned long long* n_out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int4 e = ent[cur_ent[i]];
    const int cb = e.z, nc = (int)((unsigned)e.w & RUN_COUNT_MASK);
    const unsigned long long o0 = atomicAdd(n_out, (unsigned long long)nc);
    for (int k = 0; k < nc; ++k) {
        const int4 c = ent[cb + k];
        const long long o = (long long)o0 + k;
        if (o >= max_nodes) break;
        parent[o] = cur_rec[i]; token[o] = c.x; count[o] = c.y; depth[o] = level;
        if ((unsigned)c.w & RUN_COUNT_MASK) {
            const int q = atomicAdd(n_next, 1);
            next_ent[q] = cb + k; next_rec[q] = (int)o;
        }
    }
}

}  // namespace

extern "C" int sd_enumerate(sd_store* s, int32_t tree, int64_t max_nodes, int32_t* d_parent, int32_t* d_token,
                            int32_t* d_count, int32_t* d_depth, int64_t* h_n, void* stream) {
    if (!s || !h_n || tree < -1 || tree >= s->R || max_nodes < 0 || max_nodes > 0x7fffffffll) return SD_ERR_INVALID_ARG;
    if (max_nodes > 0 && (!d_parent || !d_token || !d_count || !d_depth)) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    cudaStream_t st = (cudaStream_t)stream;
    const int4* ent = tree < 0 ? s->g_ent : s->s_ent + (long long)tree * s->spn;
    const int32_t* root = tree < 0 ? s->g_root : s->s_root + (long long)tree * s->V;
    *h_n = 0;
    const long long room = max_nodes > 0 ? max_nodes : 1;        // nodes with children among the records written
    int *fe[2] = {nullptr, nullptr}, *fr[2] = {nullptr, nullptr};
    unsigned char* small = nullptr;                              // n_out, frontier sizes
    bool okm = cudaMalloc(&small, 64) == cudaSuccess;
    for (int b = 0; b < 2 && okm; ++b)
        okm = cudaMalloc(&fe[b], sizeof(int) * (size_t)room) == cudaSuccess && cudaMalloc(&fr[b], sizeof(int) * (size_t)room) == cudaSuccess;
    auto release = [&]() { cudaFree(small); for (int b = 0; b < 2; ++b) { cudaFree(fe[b]); cudaFree(fr[b]); } };
    if (!okm) { cudaGetLastError(); release(); return SD_ERR_NOMEM; }
    unsigned long long* n_out = (unsigned long long*)small;
    int* cnt = (int*)(small + 8);                                // cnt[0], cnt[1]: frontier sizes
    cudaError_t ce = cudaMemsetAsync(small, 0, 64, st);
    enumerate_root_kernel<<<(s->V + 255) / 256, 256, 0, st>>>(ent, root, s->V, max_nodes, d_parent, d_token, d_count, d_depth,
                                                             fe[0], fr[0], cnt, n_out);
    int n = 0, cur = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&n, cnt, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    for (int level = 2; ce == cudaSuccess && n > 0 && level <= SD_MAX_DEPTH; ++level) {
        ce = cudaMemsetAsync(cnt + (cur ^ 1), 0, sizeof(int), st);
        enumerate_level_kernel<<<(n + 255) / 256, 256, 0, st>>>(ent, fe[cur], fr[cur], n, level, max_nodes, d_parent, d_token,
                                                               d_count, d_depth, fe[cur ^ 1], fr[cur ^ 1], cnt + (cur ^ 1), n_out);
        if (ce == cudaSuccess) ce = cudaMemcpyAsync(&n, cnt + (cur ^ 1), sizeof(int), cudaMemcpyDeviceToHost, st);
        if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
        cur ^= 1;
    }
    unsigned long long total = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&total, n_out, sizeof(total), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce == cudaSuccess) ce = cudaGetLastError();
    release();
    if (ce != cudaSuccess) return SD_ERR_CUDA;
    *h_n = (int64_t)total;
    return (long long)total > max_nodes ? SD_ERR_CAPACITY : SD_OK;
}
