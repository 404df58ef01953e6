// Read-only queries on a store: COUNT of token paths (the quantity Eq. 1 divides), per-slot and
// store-wide bookkeeping, empirical entropy.  The global tree is walked through its entries; a
// per-request tree is its text (common.cuh), so its counts are numbers of occurrences in the text.
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
    if (tree == -1 && len >= 1 && len <= sv.D) {
        const int4* ent = sv.g_ent;
        int x = d_paths[b];
        int node = (x >= 0 && x < sv.V) ? sv.g_root[x] : -1;
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
    } else if (tree >= 0 && tree < sv.R && len >= 1 && len <= sv.D) {
        // occurrences of the path in the request's text
        const int32_t* text = sv.s_text + (long long)tree * sv.Tp;
        const int t = sv.s_state[tree].len;
        const int x0 = d_paths[b];
        for (int s = 0; s + len <= t; ++s) {
            if (text[s] != x0) continue;
            int k = 1;
            while (k < len && text[s + k] == d_paths[b + k]) ++k;
            count += k == len ? 1 : 0;
        }
    }
    d_counts[i] = count;
}

__global__ void slot_info_kernel(sd_store sv, int n, const int32_t* d_slot, int32_t* d_len, int32_t* d_nodes,
                                 int32_t* d_status) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int slot = d_slot[i];
    int len = 0, status = SD_STATUS_BAD_SLOT;
    if (slot >= 0 && slot < sv.R) {
        const SlotState* ss = sv.s_state + slot;
        len = ss->len; status = ss->status;
    }
    if (d_len) d_len[i] = len;
    if (d_nodes) d_nodes[i] = 0;                                 // slot_nodes_kernel adds the nodes up
    if (d_status) d_status[i] = status;
}

// Nodes of a per-request tree = distinct substrings of at most D tokens of its text.  Every one
// is counted at its first occurrence: start position s brings min(D, t - s) strings, of which
// those no longer than its longest common prefix with an earlier start are not new.
// Grid: (chunks of 256 start positions, requests).
__global__ void slot_nodes_kernel(sd_store sv, const int32_t* d_slot, int32_t* d_nodes) {
    const int slot = d_slot[blockIdx.y];
    if (slot < 0 || slot >= sv.R) return;
    const int32_t* text = sv.s_text + (long long)slot * sv.Tp;
    const int t = sv.s_state[slot].len;
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    int fresh = 0;
    if (s < t) {
        const int L = min(sv.D, t - s);
        const int x0 = text[s];
        int seen = 0;                                            // longest common prefix with an earlier start
        for (int j = 0; j < s && seen < L; ++j) {
            if (text[j] != x0) continue;
            int k = 1;
            while (k < L && text[j + k] == text[s + k]) ++k;
            seen = max(seen, k);
        }
        fresh = L - seen;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) fresh += __shfl_xor_sync(0xffffffffu, fresh, o);
    if ((threadIdx.x & 31) == 0 && fresh) atomicAdd(&d_nodes[blockIdx.y], fresh);
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
    if (!d_slot || n > 65535) return SD_ERR_INVALID_ARG;
    slot_info_kernel<<<(unsigned)((n + 127) / 128), 128, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_len, d_nodes,
                                                                                  d_status);
    if (d_nodes)
        slot_nodes_kernel<<<dim3((unsigned)((s->T + 255) / 256), (unsigned)n), 256, 0, (cudaStream_t)stream>>>(*s, d_slot, d_nodes);
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
    out->slot_pool_nodes = 0;
    out->device_bytes = s->device_bytes;
    out->global_status = g.status;
    return SD_OK;
}

// ---------------------------------------------------------------------------------------------
// Empirical entropy of a tree (Appendix "Predicting SuffixDecoding Effectiveness"): for every
// node the entropy of its children's count distribution, averaged over the nodes with the
// sibling sum as weight.  With S the sum of a node's children's counts c, S times its entropy
// is  S log2 S - sum c log2 c.  Global tree: level-by-level traversal from the root table (the
// pool also holds abandoned runs and top-block copies, so a plain sweep would count too much).
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

// A per-request tree, from its text.  Thread s looks at the strings that start at position s: for
// every length L it knows their COUNT c (starts whose common prefix with s is at least L) and
// whether s is the first start of that string, in which case the string is a node and
// contributes  -c log2 c  as a child of its parent and, if it is shorter than D,  S log2 S  as a
// parent, S = c minus the occurrence that ends the text (sum of its children's counts).
__global__ void entropy_text_kernel(sd_store sv, int slot, double* acc, unsigned long long* wsum) {
    const int32_t* text = sv.s_text + (long long)slot * sv.Tp;
    const int t = sv.s_state[slot].len;
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    double part = 0.0;
    unsigned long long S_total = 0;
    if (s < t) {
        const int L = min(sv.D, t - s);
        int hist[SD_MAX_DEPTH + 1];                              // hist[k]: other starts with common prefix exactly k
        unsigned long long ends = 0;                                     // bit L: an occurrence of the L-token string ends the text
#pragma unroll
        for (int k = 0; k <= SD_MAX_DEPTH; ++k) hist[k] = 0;
        const int x0 = text[s];
        int seen = 0;
        for (int j = 0; j < t; ++j) {
            int k = 0;
            if (j != s) {
                if (text[j] != x0) continue;
                const int lim = min(L, t - j);
                k = 1;
                while (k < lim && text[j + k] == text[s + k]) ++k;
                hist[k] += 1;
                if (j < s) seen = max(seen, k);
            } else {
                k = L;
            }
            if (t - j <= k && t - j <= L) ends |= 1ull << (t - j);  // the match reaches the end of the text
        }
        int c = 1;                                               // this start itself
        for (int len = L; len >= 1; --len) {
            c += hist[len];                                      // starts that share at least `len` tokens
            if (len > seen) {                                    // first occurrence: a node
                const double dc = (double)c;
                part -= dc * log2(dc);
                if (len < sv.D) {
                    const int S = c - (int)((ends >> len) & 1ull);
                    if (S > 0) { part += (double)S * log2((double)S); S_total += (unsigned long long)S; }
                }
            }
        }
    }
    if (s == 0 && t > 0) { part += (double)t * log2((double)t); S_total += (unsigned long long)t; }   // the root
    warp_accumulate(part, S_total, acc, wsum);
}

}  // namespace

static int entropy_of_text(sd_store* s, int32_t slot, double* h_entropy, cudaStream_t st) {
    SlotState ss;
    SD_CUDA_OK(cudaMemcpyAsync(&ss, s->s_state + slot, sizeof(ss), cudaMemcpyDeviceToHost, st));
    SD_CUDA_OK(cudaStreamSynchronize(st));
    *h_entropy = 0.0;
    if (ss.len <= 0) return SD_OK;
    unsigned char* small = nullptr;
    if (cudaMalloc(&small, 64) != cudaSuccess) { cudaGetLastError(); return SD_ERR_NOMEM; }
    double* acc = (double*)small;
    unsigned long long* wsum = (unsigned long long*)(small + 8);
    cudaError_t ce = cudaMemsetAsync(small, 0, 64, st);
    entropy_text_kernel<<<(unsigned)((ss.len + 127) / 128), 128, 0, st>>>(*s, slot, acc, wsum);
    double h_acc = 0.0;
    unsigned long long h_w = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_acc, acc, sizeof(double), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_w, wsum, sizeof(h_w), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    cudaFree(small);
    if (ce != cudaSuccess) return SD_ERR_CUDA;
    *h_entropy = h_w ? h_acc / (double)h_w : 0.0;
    return SD_OK;
}

extern "C" int sd_entropy(sd_store* s, int32_t tree, double* h_entropy, void* stream) {
    if (!s || !h_entropy || tree < -1 || tree >= s->R) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    cudaStream_t st = (cudaStream_t)stream;
    if (tree >= 0) return entropy_of_text(s, tree, h_entropy, st);
    const int4* ent = s->g_ent;
    const int32_t* root = s->g_root;
    int live = 0;
    {
        GlobalState g;
        SD_CUDA_OK(cudaMemcpyAsync(&g, s->g_state, sizeof(g), cudaMemcpyDeviceToHost, st));
        SD_CUDA_OK(cudaStreamSynchronize(st));
        live = g.live;
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
