// Offline build of the global suffix tree (Section 3, "Suffix Tree Construction")
// on the GPU: depth-capped suffix sort by prefix doubling, adjacent-suffix LCPs,
// then all depths at once: ballot scans over (lcp, len) give every node's rank, range
// and parent, and one kernel lays the nodes down as sorted child runs in pre-order.
// Hand-written LSD radix sort and scans (no CUB / Thrust).
// Also: sd_build_requests (the trees of a batch of new requests by the same pipeline).
#include <algorithm>
#include <new>
#include <stdio.h>
#include <string.h>

#include "common.cuh"

namespace {

typedef unsigned long long u64;
typedef long long i64;

// ------------------------------------------------------------------ scan
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = 8;
constexpr int SCAN_TILE = SCAN_THREADS * SCAN_ITEMS;

struct LoadInt {
    const int* p;
    __device__ int operator()(i64 i) const { return p[i]; }
};

// Exclusive scan inside each tile of 2048 values f(i); tile totals go to sums[].
template <class F>
__global__ void scan_tiles_kernel(F f, i64 n, int* out, int* sums) {
    __shared__ int wsum[SCAN_THREADS / 32];
    const i64 base = (i64)blockIdx.x * SCAN_TILE + (i64)threadIdx.x * SCAN_ITEMS;
    int v[SCAN_ITEMS];
    int s = 0;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        i64 idx = base + k;
        v[k] = idx < n ? f(idx) : 0;
        s += v[k];
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int inc = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    if (lane == 31) wsum[w] = inc;
    __syncthreads();
    if (w == 0) {
        int x = lane < SCAN_THREADS / 32 ? wsum[lane] : 0;
        int xi = x;
#pragma unroll
        for (int o = 1; o < SCAN_THREADS / 32; o <<= 1) {
            int y = __shfl_up_sync(0xffffffffu, xi, o);
            if (lane >= o) xi += y;
        }
        if (lane < SCAN_THREADS / 32) wsum[lane] = xi - x;
        if (lane == SCAN_THREADS / 32 - 1) sums[blockIdx.x] = xi;
    }
    __syncthreads();
    int ex = wsum[w] + inc - s;
#pragma unroll
    for (int k = 0; k < SCAN_ITEMS; ++k) {
        i64 idx = base + k;
        if (idx < n) out[idx] = ex;
        ex += v[k];
    }
}

__global__ void scan_add_kernel(int* out, i64 n, const int* tile_offsets) {
    const i64 base = (i64)blockIdx.x * SCAN_TILE;
    const int add = tile_offsets[blockIdx.x];
    for (int k = threadIdx.x; k < SCAN_TILE; k += SCAN_THREADS) {
        i64 idx = base + k;
        if (idx < n) out[idx] += add;
    }
}

// Second half of a two-launch scan for up to 1024 tiles: every block adds up the totals of the
// tiles before it by itself (a block-wide reduction over at most 1024 numbers), so the tile
// totals need no scan of their own.  The last block also writes the grand total.
__global__ void scan_add_direct_kernel(int* out, i64 n, const int* sums, int nb, int* total_out) {
    __shared__ int wpart[SCAN_THREADS / 32];
    __shared__ int offset_sh, total_sh;
    int before = 0, all = 0;
    for (int k = threadIdx.x; k < nb; k += SCAN_THREADS) {
        const int v = sums[k];
        all += v;
        if (k < (int)blockIdx.x) before += v;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        before += __shfl_xor_sync(0xffffffffu, before, o);
        all += __shfl_xor_sync(0xffffffffu, all, o);
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) wpart[w] = before;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int k = 0; k < SCAN_THREADS / 32; ++k) t += wpart[k];
        offset_sh = t;
    }
    __syncthreads();
    if (lane == 0) wpart[w] = all;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int k = 0; k < SCAN_THREADS / 32; ++k) t += wpart[k];
        total_sh = t;
    }
    __syncthreads();
    const int add = offset_sh;
    const i64 base = (i64)blockIdx.x * SCAN_TILE;
    for (int k = threadIdx.x; k < SCAN_TILE; k += SCAN_THREADS) {
        const i64 idx = base + k;
        if (idx < n) out[idx] += add;
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) *total_out = total_sh;
}

inline i64 scan_tmp_ints(i64 n) {       // ints of scratch exclusive_scan() needs
    i64 total = 0;
    while (true) {
        i64 nb = (n + SCAN_TILE - 1) / SCAN_TILE;
        if (nb < 1) nb = 1;
        total += (nb + 31) / 32 * 32;
        if (nb == 1) break;
        n = nb;
    }
    return total + 32;
}

// In-place exclusive scan of data[0..n); grand total to *total_out.
void scan_in_place(int* data, i64 n, int* tmp, int* total_out, cudaStream_t st) {
    i64 nb = (n + SCAN_TILE - 1) / SCAN_TILE;
    if (nb < 1) nb = 1;
    scan_tiles_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(LoadInt{data}, n, data, tmp);
    if (nb <= 1024) {
        scan_add_direct_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(data, n, tmp, (int)nb, total_out);
    } else {
        scan_in_place(tmp, nb, tmp + (nb + 31) / 32 * 32, total_out, st);
        scan_add_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(data, n, tmp);
    }
}

// out[i] = sum_{k<i} f(k) for i in [0, n]; out has n + 1 slots.
template <class F>
void exclusive_scan(F f, i64 n, int* out, int* tmp, cudaStream_t st) {
    i64 nb = (n + SCAN_TILE - 1) / SCAN_TILE;
    if (nb < 1) nb = 1;
    scan_tiles_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(f, n, out, tmp);
    if (nb <= 1024) {
        scan_add_direct_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(out, n, tmp, (int)nb, out + n);
    } else {
        scan_in_place(tmp, nb, tmp + (nb + 31) / 32 * 32, out + n, st);
        scan_add_kernel<<<(unsigned)nb, SCAN_THREADS, 0, st>>>(out, n, tmp);
    }
}

// ------------------------------------------------------------------ radix sort
constexpr int RS_THREADS = 256;
constexpr int RS_ITEMS = 8;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;

__global__ void rs_hist_kernel(const u64* keys, i64 n, int shift, int* hist, int nblk) {
    __shared__ int h[256];
    h[threadIdx.x] = 0;
    __syncthreads();
    const i64 base = (i64)blockIdx.x * RS_TILE;
    for (int k = threadIdx.x; k < RS_TILE; k += RS_THREADS) {
        i64 idx = base + k;
        if (idx < n) atomicAdd(&h[(int)((keys[idx] >> shift) & 255)], 1);
    }
    __syncthreads();
    hist[(i64)threadIdx.x * nblk + blockIdx.x] = h[threadIdx.x];
}

// Stable scatter of one 8-bit digit.  offsets[d * nblk + b] is the first output
// slot of digit d for tile b.
__global__ void rs_scatter_kernel(const u64* keys_in, const uint32_t* vals_in, u64* keys_out,
                                  uint32_t* vals_out, i64 n, int shift, const int* offsets, int nblk) {
    __shared__ int warp_cnt[RS_THREADS / 32][256];
    __shared__ int base[256];
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    base[tid] = offsets[(i64)tid * nblk + blockIdx.x];
    const i64 tile0 = (i64)blockIdx.x * RS_TILE;
    for (int r = 0; r < RS_ITEMS; ++r) {
#pragma unroll
        for (int ww = 0; ww < RS_THREADS / 32; ++ww) warp_cnt[ww][tid] = 0;
        __syncthreads();
        const i64 idx = tile0 + (i64)r * RS_THREADS + tid;
        const bool valid = idx < n;
        u64 key = 0;
        uint32_t val = 0;
        int digit = 256 + lane;                       // unique: matches nobody
        if (valid) {
            key = keys_in[idx];
            val = vals_in[idx];
            digit = (int)((key >> shift) & 255);
        }
        const unsigned peers = __match_any_sync(0xffffffffu, digit);
        const int rank_in_warp = __popc(peers & ((1u << lane) - 1u));
        if (valid && rank_in_warp == 0) warp_cnt[w][digit] = __popc(peers);
        __syncthreads();
        {
            int run = base[tid];
#pragma unroll
            for (int ww = 0; ww < RS_THREADS / 32; ++ww) {
                int c = warp_cnt[ww][tid];
                warp_cnt[ww][tid] = run;
                run += c;
            }
            base[tid] = run;
        }
        __syncthreads();
        if (valid) {
            const int dst = warp_cnt[w][digit] + rank_in_warp;
            keys_out[dst] = key;
            vals_out[dst] = val;
        }
        __syncthreads();
    }
}

struct SortBuffers {
    u64* keys[2];
    uint32_t* vals[2];
    int* hist;        // 256 * nblk + 1
    int* scan_tmp;
};

// Sorts by the bit ranges [0, bits_lo) and [32, 32 + bits_hi) of the key, LSD.
// Input in buffer 0; returns the index of the buffer that holds the result.
int radix_sort_pairs(SortBuffers& b, i64 n, int bits_lo, int bits_hi, cudaStream_t st) {
    int cur = 0;
    const int nblk = (int)((n + RS_TILE - 1) / RS_TILE);
    if (nblk == 0) return 0;
    int shifts[16];
    int ns = 0;
    for (int s = 0; s < bits_lo; s += 8) shifts[ns++] = s;
    for (int s = 0; s < bits_hi; s += 8) shifts[ns++] = 32 + s;
    for (int k = 0; k < ns; ++k) {
        rs_hist_kernel<<<nblk, RS_THREADS, 0, st>>>(b.keys[cur], n, shifts[k], b.hist, nblk);
        scan_in_place(b.hist, (i64)256 * nblk, b.scan_tmp, b.hist + (i64)256 * nblk, st);
        rs_scatter_kernel<<<nblk, RS_THREADS, 0, st>>>(b.keys[cur], b.vals[cur], b.keys[cur ^ 1], b.vals[cur ^ 1],
                                                       n, shifts[k], b.hist, nblk);
        cur ^= 1;
    }
    return cur;
}

// ------------------------------------------------------------------ suffix order
// end_pos[i]: one past the last token of the sequence that holds position i.
__global__ void seq_end_kernel(const int64_t* seq_offsets, int n_seqs, i64 n, int* end_pos) {
    i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    int lo = 0, hi = n_seqs;                          // largest s with seq_offsets[s] <= i
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (seq_offsets[mid] <= i) lo = mid; else hi = mid;
    }
    end_pos[i] = (int)seq_offsets[lo + 1];
}

// bad[0] != 0 when a token is outside [0, V) or the offsets do not ascend from 0
__global__ void validate_kernel(const int32_t* tok, i64 n, int V, const int64_t* seq_offsets, int n_seqs, int* bad) {
    i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n && (tok[i] < 0 || tok[i] >= V)) atomicOr(bad, 1);
    if (i < n_seqs && seq_offsets[i] > seq_offsets[i + 1]) atomicOr(bad, 2);
    if (i == 0 && seq_offsets[0] != 0) atomicOr(bad, 2);
}

__global__ void rank0_kernel(const int32_t* tok, i64 n, int* rank) {
    i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) rank[i] = tok[i] + 1;                  // 0 is "past the end of the sequence"
}

// key = (rank of the first `off` tokens, rank of the next block) ; 0 pads short suffixes
__global__ void make_keys_kernel(const int* ra, const int* rb, int off, const int* end_pos, i64 n, u64* keys,
                                 uint32_t* vals) {
    i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    unsigned second = (i + off < end_pos[i]) ? (unsigned)rb[i + off] : 0u;
    keys[i] = ((u64)(unsigned)ra[i] << 32) | second;
    vals[i] = (uint32_t)i;
}

struct KeyChange {
    const u64* keys;
    __device__ int operator()(i64 j) const { return j == 0 ? 1 : (keys[j] != keys[j - 1] ? 1 : 0); }
};

__global__ void assign_rank_kernel(const u64* keys, const uint32_t* vals, const int* ex, i64 n, int* rank_out) {
    i64 j = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    int flag = j == 0 ? 1 : (keys[j] != keys[j - 1] ? 1 : 0);
    rank_out[vals[j]] = ex[j] + flag;                 // dense, 1-based
}

// Suffix order of sequences that are sorted one by one (the trees of different requests share
// nothing, so no suffix of one request is ever compared with a suffix of another): one block per
// sequence, tokens and suffix indices in shared memory, bitonic sort with a comparison of at most
// D tokens.  Order: by the first D tokens, a suffix that ends earlier before its extensions, equal
// strings by position, which is the order the prefix-doubling rounds produce.  One launch instead of
// about a hundred, which is what counts when a few prompts are built in the middle of a decode loop.
constexpr int BS_THREADS = 1024;
constexpr int BS_MAX_LEN = 16384;              // longest sequence (2 x 64 KB of shared memory)

__global__ void __launch_bounds__(BS_THREADS)
block_suffix_sort_kernel(const int32_t* tok, const int64_t* seq_off, int D, uint32_t* sa) {
    extern __shared__ int bs_smem[];
    const i64 b = seq_off[blockIdx.x], e = seq_off[blockIdx.x + 1];
    const int n = (int)(e - b), tid = threadIdx.x;
    if (n <= 0) return;
    int np = 1;
    while (np < n) np <<= 1;
    int* t = bs_smem;                          // [n] tokens
    int* idx = bs_smem + n;                    // [np] suffixes (>= n: padding, sorts last)
    for (int i = tid; i < n; i += BS_THREADS) t[i] = tok[b + i];
    for (int i = tid; i < np; i += BS_THREADS) idx[i] = i;
    __syncthreads();
    auto less = [&](int a, int c) -> bool {    // strict total order, a != c
        if (a >= n || c >= n) return a < c;
        const int la = min(D, n - a), lc = min(D, n - c), m = min(la, lc);
        for (int l = 0; l < m; ++l) {
            const int x = t[a + l], y = t[c + l];
            if (x != y) return x < y;
        }
        if (la != lc) return la < lc;
        return a < c;
    };
    for (int k = 2; k <= np; k <<= 1)
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int q = tid; q < (np >> 1); q += BS_THREADS) {
                const int i = ((q & ~(j - 1)) << 1) | (q & (j - 1)), p = i | j;
                const int a = idx[i], c = idx[p];
                const bool up = (i & k) == 0;
                if (less(c, a) == up) { idx[i] = c; idx[p] = a; }
            }
            __syncthreads();
        }
    for (int i = tid; i < n; i += BS_THREADS) sa[b + i] = (uint32_t)(b + idx[i]);
}

// lcp[j] = common prefix (capped) of sorted suffixes j-1 and j; len[j] = capped length of suffix j
__global__ void lcp_kernel(const int32_t* tok, const uint32_t* sa, const int* end_pos, i64 n, int D, uint8_t* lcp,
                           uint8_t* len) {
    i64 j = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    i64 b = sa[j];
    int lb = min((i64)D, (i64)end_pos[b] - b);
    len[j] = (uint8_t)lb;
    int l = 0;
    if (j > 0) {
        i64 a = sa[j - 1];
        int la = min((i64)D, (i64)end_pos[a] - a);
        int m = min(la, lb);
        while (l < m && tok[a + l] == tok[b + l]) ++l;
    }
    lcp[j] = (uint8_t)l;
}

struct NewNodes {             // nodes opened by suffix j: one at every depth in (lcp[j], len[j]]
    const uint8_t* lcp;
    const uint8_t* len;
    __device__ int operator()(i64 j) const { return (int)len[j] - (int)lcp[j]; }
};

// ------------------------------------------------------------------ all depths at once
// Everything the tree needs beyond the suffix order follows from lcp[] and len[], for all
// depths d = 1 .. D together.  "Channel" c stands for depth d = c + 1:
//   opens_c(i)  = lcp[i] <= c < len[i]    suffix i opens a node at depth d
//   bound_c(i)  = lcp[i] <= c             suffix i starts a new range of equal d-token prefixes
//   E_c[j]      = #{ i < j : opens_c(i) }                  rank of a depth-d node among all of them
//   end(j, d)   = min{ i > j : bound_c(i) } (else N)        one past the node's range: count = end - j
//   before(j)   = max{ i < j : lcp[i] < lcp[j] }            first suffix of the parent's range when
//                                                           the parent was opened by another suffix
// One warp scans a tile of 32 x CHUNKS suffixes, 32 at a time: a ballot per channel turns the 32
// suffixes' flags into one word, lane c keeps the running state of channel c.  Three launches:
// tile totals, carries across tiles (one small block), then the tile again with its carries.
// Nodes are numbered in depth-first pre-order: the root is 0 and the node that suffix j opens
// at depth d is 1 + nbase[j] + (d - lcp[j] - 1).  Pre-order is what makes paths contiguous:
// child runs are laid down in node order, so the run of a node's first child directly follows
// the node's own run, and a chain of only children is one run of consecutive entries.
constexpr int MS_CHUNKS = 32;                     // chunks of 32 suffixes per tile
constexpr int MS_CHUNKS_SMALL = 4;                // ... when there are few suffixes (more, shorter tiles: more warps at work)
constexpr i64 MS_SMALL_N = 1 << 17;
constexpr int MS_WARPS = 4;                       // tiles (warps) per block

struct LevelTables {
    int* E;               // [D][N + 1]
    int* node_end;        // [n_nodes + 1], by node id
    int* before;          // [N]
    int* agg;             // [3][32][tiles]: opens counts, last bound index, first bound index, per channel
    i64 N;
    int D, tiles;
};

template <int CHUNKS>
__global__ void __launch_bounds__(MS_WARPS * 32)
ms_tile_kernel(const uint8_t* __restrict__ lcp, const uint8_t* __restrict__ len, LevelTables T) {
    const int lane = threadIdx.x & 31;
    const int tile = blockIdx.x * MS_WARPS + (threadIdx.x >> 5);
    if (tile >= T.tiles) return;
    const i64 t0 = (i64)tile * (32 * CHUNKS);
    int cnt = 0, last = -1, first = 0x7fffffff;                 // of channel `lane`
    for (int ch = 0; ch < CHUNKS; ++ch) {
        const i64 base = t0 + (i64)ch * 32, i = base + lane;
        const int l = i < T.N ? lcp[i] : 255, n = i < T.N ? len[i] : 0;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const unsigned ob = __ballot_sync(0xffffffffu, l <= c && c < n);
            const unsigned bb = __ballot_sync(0xffffffffu, l <= c);
            if (lane == c) {
                cnt += __popc(ob);
                if (bb) {
                    last = (int)base + 31 - __clz(bb);
                    if (first == 0x7fffffff) first = (int)base + __ffs(bb) - 1;
                }
            }
        }
    }
    T.agg[(i64)lane * T.tiles + tile] = cnt;
    T.agg[(i64)(32 + lane) * T.tiles + tile] = last;
    T.agg[(i64)(64 + lane) * T.tiles + tile] = first;
}

// In place: counts -> sum over the tiles before; last -> nearest bound index before the tile
// (-1: none); first -> nearest bound index behind the tile (N: none).  Also E_c[N].
// One block per column (kind, channel) of agg[96][tiles]; every thread takes a contiguous
// stretch of tiles, the stretches' totals are combined in shared memory.
constexpr int MC_THREADS = 256;
__global__ void __launch_bounds__(MC_THREADS) ms_carry_kernel(LevelTables T) {
    __shared__ int part[MC_THREADS];
    const int kind = blockIdx.x >> 5, c = blockIdx.x & 31;
    int* col = T.agg + (i64)blockIdx.x * T.tiles;
    const int per = (T.tiles + MC_THREADS - 1) / MC_THREADS;
    // kind 2 runs over the tiles from the last to the first
    const int ident = kind == 0 ? 0 : (kind == 1 ? -1 : (int)T.N);
    auto at = [&](int k) { return kind == 2 ? T.tiles - 1 - k : k; };
    auto op = [&](int x, int y) { return kind == 0 ? x + y : (kind == 1 ? max(x, y) : min(x, y)); };
    const int k0 = threadIdx.x * per, k1 = min(T.tiles, k0 + per);
    int acc = ident;
    for (int k = k0; k < k1; ++k) acc = op(acc, col[at(k)]);
    part[threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = ident;
        for (int t = 0; t < MC_THREADS; ++t) { const int v = part[t]; part[t] = run; run = op(run, v); }
        if (kind == 0 && c < T.D) T.E[(i64)c * (T.N + 1) + T.N] = run;
    }
    __syncthreads();
    int run = part[threadIdx.x];
    for (int k = k0; k < k1; ++k) { const int v = col[at(k)]; col[at(k)] = run; run = op(run, v); }
}

template <int CHUNKS>
__global__ void __launch_bounds__(MS_WARPS * 32)
ms_apply_kernel(const uint8_t* __restrict__ lcp, const uint8_t* __restrict__ len, const int* __restrict__ nbase,
                LevelTables T) {
    __shared__ unsigned bmask[MS_WARPS][CHUNKS][32];            // bound words of the tile, by chunk and channel
    __shared__ int sfirst[MS_WARPS][32];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int tile = blockIdx.x * MS_WARPS + wib;
    if (tile >= T.tiles) return;
    const i64 t0 = (i64)tile * (32 * CHUNKS);
    const unsigned lt = (1u << lane) - 1u;
    int run_cnt = T.agg[(i64)lane * T.tiles + tile], run_last = T.agg[(i64)(32 + lane) * T.tiles + tile],
        run_first = T.agg[(i64)(64 + lane) * T.tiles + tile];
    // forward: E and `before`
    for (int ch = 0; ch < CHUNKS; ++ch) {
        const i64 base = t0 + (i64)ch * 32, i = base + lane;
        const int l = i < T.N ? lcp[i] : 255, n = i < T.N ? len[i] : 0;
        const int prev_last = run_last;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            const unsigned ob = __ballot_sync(0xffffffffu, l <= c && c < n);
            const unsigned bb = __ballot_sync(0xffffffffu, l <= c);
            const int carry = __shfl_sync(0xffffffffu, run_cnt, c);
            if (c < T.D && i < T.N) T.E[(i64)c * (T.N + 1) + i] = carry + __popc(ob & lt);
            if (lane == c) {
                run_cnt += __popc(ob);
                if (bb) run_last = (int)base + 31 - __clz(bb);
                bmask[wib][ch][c] = bb;
            }
        }
        __syncwarp();
        // nearest earlier suffix with a smaller lcp: bound channel lcp - 1
        const int src = (l >= 1 && l <= 32) ? l - 1 : 0;
        const int far = __shfl_sync(0xffffffffu, prev_last, src);
        if (i < T.N) {
            int b = -1;
            if (l >= 1) {
                const unsigned m = bmask[wib][ch][src] & lt;
                b = m ? (int)base + 31 - __clz(m) : far;
            }
            T.before[i] = b;
        }
    }
    // backward: the end of every node's range
    for (int ch = CHUNKS - 1; ch >= 0; --ch) {
        const i64 base = t0 + (i64)ch * 32, i = base + lane;
        sfirst[wib][lane] = run_first;
        __syncwarp();
        if (i < T.N) {
            const int l = lcp[i], n = len[i];
            const unsigned gt = ~lt & ~(1u << lane);
            int nid = 1 + nbase[i];
            for (int d = l + 1; d <= n; ++d, ++nid) {
                const unsigned m = bmask[wib][ch][d - 1] & gt;
                T.node_end[nid] = m ? (int)base + __ffs(m) - 1 : sfirst[wib][d - 1];
            }
        }
        __syncwarp();
        const unsigned bb = bmask[wib][ch][lane];
        if (bb) run_first = (int)base + __ffs(bb) - 1;
    }
}

// children per node: the depth d + 1 nodes opened inside the node's range
__global__ void count_children_kernel(const uint8_t* __restrict__ lcp, const uint8_t* __restrict__ len,
                                      const int* __restrict__ nbase, LevelTables T, int* nchild) {
    const i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) nchild[0] = T.E[T.N];                            // the root's children: all depth-1 nodes
    if (i >= T.N) return;
    const int l = lcp[i], n = len[i];
    int nid = 1 + nbase[i];
    for (int d = l + 1; d <= n; ++d, ++nid) {
        int nc = 0;
        if (d < T.D) {
            const int* row = T.E + (i64)d * (T.N + 1);          // channel of depth d + 1
            nc = row[T.node_end[nid]] - row[i];
        }
        nchild[nid] = nc;
    }
}

__device__ __forceinline__ int top_block_of(int nid, int nc) { return (nid > 0 && nc > SD_TOP_MIN) ? SD_TOP_BLOCK : 0; }

struct RunAlloc {             // entries a node's child run takes, top block included
    const int* nchild;
    int top_blocks;
    __device__ int operator()(i64 nid) const {
        return nchild[nid] + (top_blocks ? top_block_of((int)nid, nchild[nid]) : 0);
    }
};

__global__ void collect_wide_kernel(const int* nchild, i64 n_nodes_plus1, int* list, int* counter) {
    i64 nid = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (nid >= n_nodes_plus1) return;
    if (top_block_of((int)nid, nchild[nid])) list[atomicAdd(counter, 1)] = (int)nid;
}

// One block per long run: header (sum of counts) and the 64 best children by (count desc,
// token asc), found by 64 rounds of "largest key below the previous one".
__global__ void fill_top_kernel(const int* list, const int* nchild, const int* runstart, int4* ent) {
    __shared__ u64 skey[256];
    __shared__ int sidx[256];
    __shared__ u64 ssum[256];
    const int nid = list[blockIdx.x];
    const int n = nchild[nid];
    const int top = runstart[nid];                 // header; the run itself starts SD_TOP_BLOCK later
    const int4* run = ent + top + SD_TOP_BLOCK;
    u64 sum = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) sum += (u64)(unsigned)run[i].y;
    ssum[threadIdx.x] = sum;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) ssum[threadIdx.x] += ssum[threadIdx.x + o];
        __syncthreads();
    }
    const int ntop = n < 64 ? n : 64;
    if (threadIdx.x == 0) ent[top] = make_int4((int)(unsigned)(ssum[0] & 0xffffffffu), (int)(unsigned)(ssum[0] >> 32), ntop, 0);
    u64 prev = ~0ull;
    for (int r = 0; r < ntop; ++r) {
        u64 best = 0;
        int bi = -1;
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            const int4 e = run[i];
            const u64 key = ((u64)(unsigned)e.y << 32) | (u64)(0xffffffffu - (unsigned)e.x);
            if (key < prev && (bi < 0 || key > best)) { best = key; bi = i; }
        }
        skey[threadIdx.x] = bi >= 0 ? best : 0;
        sidx[threadIdx.x] = bi;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if (threadIdx.x < o) {
                const int oi = sidx[threadIdx.x + o];
                if (oi >= 0 && (sidx[threadIdx.x] < 0 || skey[threadIdx.x + o] > skey[threadIdx.x])) {
                    skey[threadIdx.x] = skey[threadIdx.x + o];
                    sidx[threadIdx.x] = oi;
                }
            }
            __syncthreads();
        }
        prev = skey[0];
        if (threadIdx.x == 0) ent[top + 1 + r] = run[sidx[0]];
        __syncthreads();
    }
}

// Write the nodes that suffix j opens.  A node's entry sits in its parent's child run at its
// rank among the siblings (suffix order = token order).  The first node a suffix opens hangs
// below a node of an earlier suffix (or the root); every further one is the only-so-far child
// of the one before it.
__global__ void emit_nodes_kernel(const int32_t* tok, const uint32_t* sa, const uint8_t* lcp, const uint8_t* len, i64 n,
                                  LevelTables T, const int* nbase, const int* nchild, const int* runstart, int4* ent,
                                  int32_t* root) {
    const i64 j = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const int l = lcp[j], m = len[j];
    if (m <= l) return;
    int nid = 1 + nbase[j];
    int pnid = 0, rank = T.E[j];                                  // depth 1: below the root
    if (l >= 1) {
        const int jx = T.before[j];                               // its first suffix opened the parent
        pnid = 1 + nbase[jx] + (l - (int)lcp[jx] - 1);
        const int* row = T.E + (i64)l * (T.N + 1);                // channel of depth l + 1
        rank = row[j] - row[jx];
    }
    const i64 text = (i64)sa[j];
    for (int d = l + 1; d <= m; ++d, ++nid) {
        const int nc = nchild[nid];
        int4 e;
        e.x = tok[text + d - 1];
        e.y = T.node_end[nid] - (int)j;                           // every suffix in the range is an occurrence
        const int tb = top_block_of(nid, nc);
        e.z = nc > 0 ? runstart[nid] + tb : 0;
        e.w = nc > 0 ? (int)((unsigned)nc | RUN_STATIC | (tb ? RUN_HAS_TOP : 0u)) : 0;
        const int pos = runstart[pnid] + top_block_of(pnid, nchild[pnid]) + rank;
        ent[pos] = e;
        if (d == 1) root[e.x] = pos;
        pnid = nid; rank = 0;
    }
}

__global__ void init_global_state_kernel(GlobalState* g, int used, int live, long long tokens) {
    g->used = used; g->live = live; g->status = 0; g->epoch = 1; g->tokens = tokens;
}

}  // namespace

// Test hook: the k-th device allocation from now on fails (k = 1: the next one); 0 switches it off.
// Only the allocation-failure tests use it.
static long long g_fail_alloc_in = 0;
static cudaError_t sd_device_malloc(void** p, size_t bytes) {
    if (g_fail_alloc_in > 0 && --g_fail_alloc_in == 0) { *p = nullptr; return cudaErrorMemoryAllocation; }
    return cudaMalloc(p, bytes);
}
extern "C" void sd_debug_fail_alloc(int64_t k) { g_fail_alloc_in = k; }

namespace {

struct DeviceArena {          // temporaries of one build: freed together, or kept in a workspace
    void* ptr[48];
    int n = 0;
    sd_workspace* keep = nullptr;                     // if set, buffers live there and are reused
    char* chunk = nullptr;                            // reserved block the next buffers are carved from
    long long chunk_left = 0;
    ~DeviceArena() { if (!keep) for (int i = 0; i < n; ++i) cudaFree(ptr[i]); }
    // One allocation for the buffers to come (an allocation of its own costs far more than the
    // kernels that use a buffer).  If it fails the buffers are simply allocated one by one.
    void reserve(long long bytes) {
        if (keep || n >= 48 || bytes <= 0) return;
        void* p = nullptr;
        if (sd_device_malloc(&p, (size_t)bytes) != cudaSuccess) { cudaGetLastError(); return; }
        ptr[n++] = p;
        chunk = (char*)p; chunk_left = bytes;
    }
    template <class T> bool get(T** out, i64 count) {
        if (count < 1) count = 1;
        const long long need = (long long)count * (long long)sizeof(T);
        const long long padded = (need + 255) / 256 * 256;
        if (!keep && chunk_left >= padded) {
            *out = (T*)chunk;
            chunk += padded; chunk_left -= padded;
            return true;
        }
        if (n >= 48) return false;
        if (keep) {
            const int k = n++;
            if (keep->bytes[k] < need) {
                if (keep->ptr[k]) cudaFree(keep->ptr[k]);
                keep->ptr[k] = nullptr; keep->bytes[k] = 0;
                const long long want = need + need / 4 + 256;
                if (sd_device_malloc(&keep->ptr[k], (size_t)want) != cudaSuccess) { cudaGetLastError(); return false; }
                keep->bytes[k] = want;
            }
            *out = (T*)keep->ptr[k];
            return true;
        }
        void* p = nullptr;
        if (sd_device_malloc(&p, (size_t)need) != cudaSuccess) { cudaGetLastError(); return false; }
        ptr[n++] = p;
        *out = (T*)p;
        return true;
    }
};

inline unsigned grid_for(i64 n, int threads) { return (unsigned)((n + threads - 1) / threads); }

int bits_for(i64 maxval) {
    int b = 1;
    while ((1ll << b) <= maxval && b < 32) ++b;
    return b;
}

}  // namespace

template <class T>
static bool store_alloc(sd_store* s, T** out, long long count) {
    void* p = nullptr;
    if (count < 1) count = 1;
    if (sd_device_malloc(&p, (size_t)count * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return false; }
    s->device_bytes += count * (long long)sizeof(T);
    *out = (T*)p;
    return true;
}

static void store_release(sd_store* s) {
    if (!s) return;
    cudaFree(s->g_ent); cudaFree(s->g_root); cudaFree(s->g_state);
    cudaFree(s->s_ent); cudaFree(s->s_root); cudaFree(s->s_text); cudaFree(s->s_state);
    if (s->ws) {
        for (int k = 0; k < 48; ++k) cudaFree(s->ws->ptr[k]);
        delete s->ws;
    }
    if (s->ev_fork) cudaEventDestroy(s->ev_fork);
    if (s->ev_join) cudaEventDestroy(s->ev_join);
    if (s->aux) cudaStreamDestroy(s->aux);
    delete s;
}

// Everything up to the placement of the child runs, for one array of sequences: suffix
// order, LCPs, children per node (pre-order node ids) and the start of every child run.
struct Pipeline {
    DeviceArena tmp;
    SortBuffers sb;
    int *end_pos = nullptr, *rank[8] = {nullptr}, *comb[2] = {nullptr, nullptr}, *ex = nullptr;
    uint8_t *lcp = nullptr, *len = nullptr;
    int* wide_counter = nullptr;
    const uint32_t* sa = nullptr;
    LevelTables lv;
    int *nbase = nullptr, *nchild = nullptr, *runstart = nullptr, *big_tmp = nullptr, *wide_list = nullptr;
    i64 N = 0, n_nodes = 0, used_entries = 0;
    int n_wide = 0;
};

// max_token: largest token value + 1 (sets the number of radix passes).  top_blocks: reserve
// room for top blocks in front of long runs.  per_seq_max_len > 0: the sequences are independent
// (tokens of different sequences never compare equal, sequence k's tokens below sequence k + 1's)
// and none is longer than that, so each is sorted by a block of its own.
// no_readback: nothing is read back to the host on the way (no stream synchronisation): the
// node arrays are sized for the most nodes N tokens can have (N * D) instead of the number
// counted, and n_nodes / used_entries / n_wide are not filled in.  For small builds without
// top blocks (a few prompts in the middle of a decode loop), where a round trip to the host
// costs as much as the kernels between two of them.
// Returns SD_OK, SD_ERR_NOMEM or SD_ERR_CUDA.
static int pipeline_run(Pipeline& P, const int32_t* d_tok, const int64_t* d_seq_offsets, int n_seqs, i64 N,
                        i64 max_token, int D, bool top_blocks, cudaStream_t st, i64 per_seq_max_len = 0,
                        bool no_readback = false) {
    const int T256 = 256;
    P.N = N;
    DeviceArena& tmp = P.tmp;
    SortBuffers& sb = P.sb;
    cudaError_t ce = cudaSuccess;
    const int nblk = (int)((N + RS_TILE - 1) / RS_TILE);
    int m = 0;
    while ((2 << m) <= D) ++m;                    // 2^m <= D < 2^(m+1)
    {
        const i64 scan_ints = scan_tmp_ints(std::max<i64>((i64)256 * nblk, N + 1));
        tmp.reserve((long long)N * (16 + 8 + 4 + 4 + 2 + 4 * (m + 1) + 8 + 4) + 4ll * ((i64)256 * nblk + 1 + scan_ints) +
                    64 * 256);
    }
    bool ok = tmp.get(&sb.keys[0], N) && tmp.get(&sb.keys[1], N) && tmp.get(&sb.vals[0], N) &&
              tmp.get(&sb.vals[1], N) && tmp.get(&sb.hist, (i64)256 * nblk + 1) &&
              tmp.get(&sb.scan_tmp, scan_tmp_ints(std::max<i64>((i64)256 * nblk, N + 1))) &&
              tmp.get(&P.end_pos, N) && tmp.get(&P.ex, N + 1) && tmp.get(&P.lcp, N) && tmp.get(&P.len, N) &&
              tmp.get(&P.wide_counter, 1);
    for (int k = 0; ok && k <= m; ++k) ok = tmp.get(&P.rank[k], N);
    ok = ok && tmp.get(&P.comb[0], N) && tmp.get(&P.comb[1], N);
    if (!ok) return SD_ERR_NOMEM;
    int *end_pos = P.end_pos, **rank = P.rank, **comb = P.comb, *ex = P.ex;
    uint8_t *lcp = P.lcp, *len = P.len;

    seq_end_kernel<<<grid_for(N, T256), T256, 0, st>>>(d_seq_offsets, n_seqs, N, end_pos);
    const bool block_sort = per_seq_max_len > 0 && per_seq_max_len <= BS_MAX_LEN;
    if (block_sort) {
        i64 np = 1;
        while (np < per_seq_max_len) np <<= 1;
        const size_t smem = (size_t)(per_seq_max_len + np) * sizeof(int);
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(block_suffix_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)((BS_MAX_LEN * 2) * sizeof(int))) != cudaSuccess)
            return SD_ERR_CUDA;
        block_suffix_sort_kernel<<<(unsigned)n_seqs, BS_THREADS, smem, st>>>(d_tok, d_seq_offsets, D, sb.vals[0]);
    } else
        rank0_kernel<<<grid_for(N, T256), T256, 0, st>>>(d_tok, N, rank[0]);
    const int bits_tok = bits_for(max_token + 1), bits_rank = bits_for(N + 1);
    int sorted = 0;
    // rank[k] orders the first 2^k tokens of every suffix
    auto round = [&](const int* ra, const int* rb, int off, int* rout) {
        make_keys_kernel<<<grid_for(N, T256), T256, 0, st>>>(ra, rb, off, end_pos, N, sb.keys[0], sb.vals[0]);
        // the token ranks of the first round need more bits than the dense ranks of the later ones
        sorted = radix_sort_pairs(sb, N, rb == rank[0] ? bits_tok : bits_rank, ra == rank[0] ? bits_tok : bits_rank, st);
        if (rout) {
            exclusive_scan(KeyChange{sb.keys[sorted]}, N, ex, sb.scan_tmp, st);
            assign_rank_kernel<<<grid_for(N, T256), T256, 0, st>>>(sb.keys[sorted], sb.vals[sorted], ex, N, rout);
        }
    };
    if (block_sort) {
        // sb.vals[0] holds the suffix order already
    } else if (m == 0) {
        round(rank[0], rank[0], 1 << 30, nullptr);        // D == 1: the first token alone
    } else {
        const bool pow2 = D == (1 << m);
        for (int k = 0; k < m; ++k)
            round(rank[k], rank[k], 1 << k, (pow2 && k == m - 1) ? nullptr : rank[k + 1]);
        if (!pow2) {
            // append the remaining binary digits of D, high to low
            int cur_len = 1 << m, rem = D - cur_len, which = 0;
            const int* cur = rank[m];
            for (int b = m - 1; b >= 0; --b) {
                if (!(rem & (1 << b))) continue;
                rem -= 1 << b;
                int* dst = rem == 0 ? nullptr : comb[which];
                round(cur, rank[b], cur_len, dst);
                cur = dst;
                which ^= 1;
                cur_len += 1 << b;
            }
        }
    }
    P.sa = sb.vals[sorted];
    lcp_kernel<<<grid_for(N, T256), T256, 0, st>>>(d_tok, P.sa, end_pos, N, D, lcp, len);
    ok = tmp.get(&P.nbase, N + 1);
    if (!ok) return SD_ERR_NOMEM;
    exclusive_scan(NewNodes{lcp, len}, N, P.nbase, sb.scan_tmp, st);
    int h_nodes = 0;
    if (!no_readback) {
        ce = cudaMemcpyAsync(&h_nodes, P.nbase + N, sizeof(int), cudaMemcpyDeviceToHost, st);
        if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
        if (ce != cudaSuccess) return SD_ERR_CUDA;
    }
    const i64 n_nodes = no_readback ? N * D : (i64)h_nodes;      // (an upper bound: every suffix opens at most D nodes)
    P.n_nodes = no_readback ? 0 : n_nodes;

    LevelTables& lv = P.lv;
    lv.N = N; lv.D = D;
    const bool small_tiles = N <= MS_SMALL_N;
    const int tile_len = 32 * (small_tiles ? MS_CHUNKS_SMALL : MS_CHUNKS);
    lv.tiles = (int)((N + tile_len - 1) / tile_len);
    tmp.reserve(4ll * ((i64)D * (N + 1) + 3 * (n_nodes + 2) + N + (i64)lv.tiles * 96 + scan_tmp_ints(n_nodes + 1) +
                       n_nodes / SD_TOP_MIN + 2) + 64 * 256);
    ok = tmp.get(&lv.E, (i64)D * (N + 1)) && tmp.get(&lv.node_end, n_nodes + 1) && tmp.get(&lv.before, N) &&
         tmp.get(&lv.agg, (i64)lv.tiles * 96) && tmp.get(&P.nchild, n_nodes + 1) &&
         tmp.get(&P.runstart, n_nodes + 2) && tmp.get(&P.big_tmp, scan_tmp_ints(n_nodes + 1)) &&
         tmp.get(&P.wide_list, n_nodes / SD_TOP_MIN + 2);
    if (!ok) return SD_ERR_NOMEM;
    const unsigned ms_grid = (unsigned)((lv.tiles + MS_WARPS - 1) / MS_WARPS);
    if (small_tiles) ms_tile_kernel<MS_CHUNKS_SMALL><<<ms_grid, MS_WARPS * 32, 0, st>>>(lcp, len, lv);
    else ms_tile_kernel<MS_CHUNKS><<<ms_grid, MS_WARPS * 32, 0, st>>>(lcp, len, lv);
    ms_carry_kernel<<<96, MC_THREADS, 0, st>>>(lv);
    if (small_tiles) ms_apply_kernel<MS_CHUNKS_SMALL><<<ms_grid, MS_WARPS * 32, 0, st>>>(lcp, len, P.nbase, lv);
    else ms_apply_kernel<MS_CHUNKS><<<ms_grid, MS_WARPS * 32, 0, st>>>(lcp, len, P.nbase, lv);
    // (with the bound, the node ids behind the last real node have no children)
    if (no_readback) ce = cudaMemsetAsync(P.nchild, 0, sizeof(int) * (size_t)(n_nodes + 1), st);
    if (ce != cudaSuccess) return SD_ERR_CUDA;
    count_children_kernel<<<grid_for(N, T256), T256, 0, st>>>(lcp, len, P.nbase, lv, P.nchild);
    // child runs (with their top blocks) in node (pre-)order
    exclusive_scan(RunAlloc{P.nchild, top_blocks ? 1 : 0}, n_nodes + 1, P.runstart, P.big_tmp, st);
    int* wide_counter = P.wide_counter;
    ce = cudaMemsetAsync(wide_counter, 0, sizeof(int), st);
    if (top_blocks)
        collect_wide_kernel<<<grid_for(n_nodes + 1, T256), T256, 0, st>>>(P.nchild, n_nodes + 1, P.wide_list, wide_counter);
    if (no_readback) return ce == cudaSuccess ? SD_OK : SD_ERR_CUDA;
    int h_total = 0;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_total, P.runstart + n_nodes + 1, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&P.n_wide, wide_counter, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) return SD_ERR_CUDA;
    P.used_entries = h_total;
    return SD_OK;
}

extern "C" int sd_build(const sd_build_params* p, const int32_t* d_corpus, const int64_t* d_seq_offsets, int32_t n_seqs,
                        void* stream, sd_store** out) {
    if (!out) return SD_ERR_INVALID_ARG;
    *out = nullptr;
    if (!p || p->vocab < 1 || p->depth_cap < 1 || p->depth_cap > SD_MAX_DEPTH || p->max_requests < 1 ||
        p->max_req_tokens < 1 || p->max_spec_cap < 1 || p->max_spec_cap > SD_MAX_SPEC || n_seqs < 0)
        return SD_ERR_INVALID_ARG;
    if (n_seqs > 0 && (!d_corpus || !d_seq_offsets)) return SD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;

    i64 N = 0;
    if (n_seqs > 0) {
        SD_CUDA_OK(cudaMemcpyAsync(&N, d_seq_offsets + n_seqs, sizeof(i64), cudaMemcpyDeviceToHost, st));
        SD_CUDA_OK(cudaStreamSynchronize(st));
        if (N < 0 || N >= (1ll << 31) - 2) return SD_ERR_INVALID_ARG;
    }

    sd_store* s = new (std::nothrow) sd_store();
    if (!s) return SD_ERR_NOMEM;
    memset(s, 0, sizeof(*s));
    s->V = p->vocab; s->D = p->depth_cap; s->R = p->max_requests; s->T = p->max_req_tokens; s->M = p->max_spec_cap;
    if (cudaGetDevice(&s->device) != cudaSuccess) { delete s; return SD_ERR_CUDA; }
    const int D = s->D;
    s->spn = p->slot_pool_nodes > 0 ? p->slot_pool_nodes : 2ll * s->T * D;
    if (s->spn >= (1ll << 31) - 2) { delete s; return SD_ERR_INVALID_ARG; }

    bool ok = store_alloc(s, &s->g_root, s->V) && store_alloc(s, &s->g_state, 1) &&
              store_alloc(s, &s->s_ent, (i64)s->R * s->spn) && store_alloc(s, &s->s_root, (i64)s->R * s->V) &&
              store_alloc(s, &s->s_text, (i64)s->R * s->T) && store_alloc(s, &s->s_state, s->R);
    if (!ok) { store_release(s); return SD_ERR_NOMEM; }
    if (cudaStreamCreateWithFlags(&s->aux, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&s->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        store_release(s);
        return SD_ERR_CUDA;
    }
    cudaError_t ce = cudaMemsetAsync(s->g_root, 0xFF, sizeof(int32_t) * (size_t)s->V, st);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(s->s_root, 0xFF, sizeof(int32_t) * (size_t)s->R * s->V, st);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(s->s_state, 0, sizeof(SlotState) * (size_t)s->R, st);
    if (ce != cudaSuccess) { store_release(s); return SD_ERR_CUDA; }

    Pipeline P;
    const int T256 = 256;
    i64 n_nodes = 0, used_entries = 0;
    if (N > 0) {
        {
            int* bad = nullptr;
            int h_bad = 0;
            if (!P.tmp.get(&bad, 1)) { store_release(s); return SD_ERR_NOMEM; }
            ce = cudaMemsetAsync(bad, 0, sizeof(int), st);
            validate_kernel<<<grid_for(std::max<i64>(N, n_seqs), T256), T256, 0, st>>>(d_corpus, N, s->V, d_seq_offsets,
                                                                                      n_seqs, bad);
            if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h_bad, bad, sizeof(int), cudaMemcpyDeviceToHost, st);
            if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
            if (ce != cudaSuccess) { store_release(s); return SD_ERR_CUDA; }
            if (h_bad) { store_release(s); return SD_ERR_INVALID_ARG; }
        }
        const int rc = pipeline_run(P, d_corpus, d_seq_offsets, n_seqs, N, s->V, D, true, st);
        if (rc != SD_OK) { store_release(s); return rc; }
        n_nodes = P.n_nodes;
        used_entries = P.used_entries;
    }

    i64 extra = p->global_extra_nodes >= 0 ? p->global_extra_nodes : std::max<i64>(1ll << 22, n_nodes);
    s->g_cap = used_entries + extra;
    if (s->g_cap >= (1ll << 31) - 2) { store_release(s); return SD_ERR_INVALID_ARG; }
    if (!store_alloc(s, &s->g_ent, s->g_cap)) { store_release(s); return SD_ERR_NOMEM; }

    if (N > 0) {
        // write the entries
        emit_nodes_kernel<<<grid_for(N, T256), T256, 0, st>>>(d_corpus, P.sa, P.lcp, P.len, N, P.lv, P.nbase, P.nchild,
                                                             P.runstart, s->g_ent, s->g_root);
        if (P.n_wide > 0) fill_top_kernel<<<P.n_wide, 256, 0, st>>>(P.wide_list, P.nchild, P.runstart, s->g_ent);
    }
    init_global_state_kernel<<<1, 1, 0, st>>>(s->g_state, (int)used_entries, (int)n_nodes, N);
    ce = cudaStreamSynchronize(st);
    if (ce == cudaSuccess) ce = cudaGetLastError();
    if (ce != cudaSuccess) { store_release(s); return SD_ERR_CUDA; }
    *out = s;
    return SD_OK;
}

extern "C" void sd_free(sd_store* s) {
    if (!s) return;
    cudaDeviceSynchronize();
    store_release(s);
}

extern "C" const char* sd_strerror(int code) {
    switch (code) {
        case SD_OK: return "ok";
        case SD_ERR_INVALID_ARG: return "invalid argument";
        case SD_ERR_CUDA: return "CUDA runtime error";
        case SD_ERR_NOMEM: return "out of device memory";
        case SD_ERR_CAPACITY: return "capacity exceeded";
        default: return "unknown error";
    }
}

// ---------------------------------------------------------------------------------------------
// sd_build_requests: the per-request trees of a batch of new requests, built from their prompts
// by the same sort-based pipeline as the global tree instead of token by token.  The prompts
// are kept apart by giving every request its own token range (token + rank * V), so one
// suffix sort orders all of them request by request and one pre-order numbering lays every
// request's nodes down contiguously; each request's part is then written into its own pool.
namespace {

__device__ __forceinline__ int seq_rank_of(const int64_t* off, int n, i64 pos) {
    int lo = 0, hi = n;                               // largest q with off[q] <= pos
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (off[mid] <= pos) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void map_tokens_kernel(const int32_t* tok, const int64_t* off, int n, i64 N, int V, int32_t* out, int* bad) {
    i64 i = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    const int t = tok[i];
    if (t < 0 || t >= V) { atomicOr(bad, 1); out[i] = 0; return; }
    out[i] = seq_rank_of(off, n, i) * V + t;
}

// one block per request: forget the slot's old tree and store the new text
__global__ void requests_prepare_kernel(sd_store sv, int n, const int32_t* slot_ids, const int64_t* off,
                                        const int32_t* tok) {
    const int q = blockIdx.x;
    if (q >= n) return;
    const int slot = slot_ids[q];
    if (slot < 0 || slot >= sv.R) return;
    SlotState* ss = sv.s_state + slot;
    int32_t* text = sv.s_text + (i64)slot * sv.T;
    int32_t* root = sv.s_root + (i64)slot * sv.V;
    const int old_len = ss->len;
    for (int k = threadIdx.x; k < old_len; k += blockDim.x) root[text[k]] = -1;
    __syncthreads();
    const i64 lo = off[q], hi = off[q + 1];
    if (hi - lo <= sv.T)
        for (i64 k = threadIdx.x; k < hi - lo; k += blockDim.x) text[k] = tok[lo + k];
}

struct RequestLayout {       // where request q's nodes go (device arrays of n entries)
    int* run_base;           // global position of its first child run
    int* n1;                 // its depth-1 nodes
    int* r1lo;               // depth-1 nodes of earlier requests
    int* used;               // entries it takes
    int* live;               // nodes
    int* ok;                 // fits its pool and text buffer
};

__global__ void requests_layout_kernel(sd_store sv, int n, const int64_t* off, const int* nbase, const int* runstart,
                                       const int* r1, RequestLayout L) {
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= n) return;
    const i64 lo = off[q], hi = off[q + 1];
    const int first = 1 + nbase[lo], next = 1 + nbase[hi];
    const int rb = runstart[first], re = runstart[next];
    const int n1 = r1[hi] - r1[lo];
    L.run_base[q] = rb; L.n1[q] = n1; L.r1lo[q] = r1[lo];
    L.used[q] = n1 + (re - rb); L.live[q] = next - first;
    L.ok[q] = ((i64)n1 + (re - rb) <= sv.spn && hi - lo <= sv.T) ? 1 : 0;
}

__global__ void emit_nodes_slots_kernel(sd_store sv, int n_req, const int32_t* slot_ids, const int64_t* off,
                                        const int32_t* mtok, const uint32_t* sa, const uint8_t* lcp, const uint8_t* len,
                                        i64 n, LevelTables T, const int* nbase, const int* nchild, const int* runstart,
                                        RequestLayout L) {
    const i64 j = (i64)blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= n) return;
    const int l = lcp[j], m = len[j];
    if (m <= l) return;
    const i64 text = (i64)sa[j];
    const int q = seq_rank_of(off, n_req, text);
    const int slot = slot_ids[q];
    if (!L.ok[q] || slot < 0 || slot >= sv.R) return;
    int4* ent = sv.s_ent + (i64)slot * sv.spn;
    const int shift = L.n1[q] - L.run_base[q];                  // global run position -> index in the slot pool
    int nid = 1 + nbase[j];
    int pos = T.E[j] - L.r1lo[q];                               // depth 1: the request's own root table
    if (l >= 1) {
        const int jx = T.before[j];
        const int pnid = 1 + nbase[jx] + (l - (int)lcp[jx] - 1);
        const int* row = T.E + (i64)l * (T.N + 1);
        pos = runstart[pnid] + (row[j] - row[jx]) + shift;
    }
    for (int d = l + 1; d <= m; ++d, ++nid) {
        const int nc = nchild[nid];
        int4 e;
        e.x = mtok[text + d - 1] - q * sv.V;
        e.y = T.node_end[nid] - (int)j;
        e.z = nc > 0 ? runstart[nid] + shift : 0;
        e.w = nc > 0 ? (int)((unsigned)nc | RUN_STATIC) : 0;
        ent[pos] = e;
        if (d == 1) (sv.s_root + (i64)slot * sv.V)[e.x] = pos;
        pos = runstart[nid] + shift;                             // the next one is this node's first child
    }
}

// one warp per request: bookkeeping and the active nodes (lane d-1: node of the last d tokens)
__global__ void requests_finalize_kernel(sd_store sv, int n, const int32_t* slot_ids, const int64_t* off,
                                         RequestLayout L) {
    const int q = (int)((blockIdx.x * (i64)blockDim.x + threadIdx.x) >> 5), lane = threadIdx.x & 31;
    if (q >= n) return;
    const int slot = slot_ids[q];
    if (slot < 0 || slot >= sv.R) return;
    SlotState* ss = sv.s_state + slot;
    const bool ok = L.ok[q] != 0;
    const int len = ok ? (int)(off[q + 1] - off[q]) : 0;
    const int4* ent = sv.s_ent + (i64)slot * sv.spn;
    const int32_t* root = sv.s_root + (i64)slot * sv.V;
    const int32_t* text = sv.s_text + (i64)slot * sv.T;
    int node = -1, rcb = 0;
    unsigned rw = 0;
    const int d = lane + 1;
    if (d <= len && d <= sv.D) {
        node = root[text[len - d]];
        int4 e = make_int4(0, 0, 0, 0);
        if (node >= 0) e = ent[node];
        for (int k = 1; k < d && node >= 0; ++k) {
            const int x = text[len - d + k];
            const int cb = e.z, nn = (int)((unsigned)e.w & RUN_COUNT_MASK);
            int lo = 0, hi = nn;
            while (lo < hi) {                                    // at most 24 rounds
                const int mid = (lo + hi) >> 1;
                if (ent[cb + mid].x < x) lo = mid + 1; else hi = mid;
            }
            node = -1;
            if (lo < nn) { e = ent[cb + lo]; if (e.x == x) node = cb + lo; }
        }
        if (node >= 0) { rcb = e.z; rw = (unsigned)e.w; }
    }
    ss->active[lane] = node; ss->room[lane] = 0; ss->run_cb[lane] = rcb; ss->run_w[lane] = rw;
    if (lane == 0) {
        ss->len = len; ss->used = ok ? L.used[q] : 0; ss->live = ok ? L.live[q] : 0;
        ss->status = ok ? 0 : SD_STATUS_POOL_FULL;
        ss->gen += 1;
    }
}

}  // namespace

extern "C" int sd_build_requests(sd_store* s, int32_t n, const int32_t* h_slot, const int64_t* h_offsets,
                                 const int32_t* d_tokens, void* stream) {
    if (!s || n < 0) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    if (n == 0) return SD_OK;
    if (!h_slot || !h_offsets || n > s->R) return SD_ERR_INVALID_ARG;
    if (h_offsets[0] != 0) return SD_ERR_INVALID_ARG;
    for (int q = 0; q < n; ++q) {
        if (h_offsets[q + 1] < h_offsets[q] || h_slot[q] < 0 || h_slot[q] >= s->R) return SD_ERR_INVALID_ARG;
        for (int r = 0; r < q; ++r) if (h_slot[r] == h_slot[q]) return SD_ERR_INVALID_ARG;   // a slot once per call
    }
    const i64 N = h_offsets[n];
    if (N > 0 && !d_tokens) return SD_ERR_INVALID_ARG;
    if ((i64)n * s->V >= (1ll << 31) - 2 || N >= (1ll << 31) - 2) return SD_ERR_CAPACITY;
    cudaStream_t st = (cudaStream_t)stream;
    const int T256 = 256, D = s->D;

    Pipeline P;
    if (!s->ws) {
        s->ws = new (std::nothrow) sd_workspace();
        if (!s->ws) return SD_ERR_NOMEM;
        memset(s->ws, 0, sizeof(*s->ws));
    }
    P.tmp.keep = s->ws;                                          // temporaries are kept for the next call
    int32_t *d_slot = nullptr, *mtok = nullptr;
    int64_t* d_off = nullptr;
    int* bad = nullptr;
    RequestLayout L;
    bool ok = P.tmp.get(&d_slot, n) && P.tmp.get(&d_off, n + 1) && P.tmp.get(&mtok, N) && P.tmp.get(&bad, 1) &&
              P.tmp.get(&L.run_base, n) && P.tmp.get(&L.n1, n) && P.tmp.get(&L.r1lo, n) &&
              P.tmp.get(&L.used, n) && P.tmp.get(&L.live, n) && P.tmp.get(&L.ok, n);
    if (!ok) return SD_ERR_NOMEM;
    SD_CUDA_OK(cudaMemcpyAsync(d_slot, h_slot, sizeof(int32_t) * n, cudaMemcpyHostToDevice, st));
    SD_CUDA_OK(cudaMemcpyAsync(d_off, h_offsets, sizeof(int64_t) * (n + 1), cudaMemcpyHostToDevice, st));
    SD_CUDA_OK(cudaMemsetAsync(bad, 0, sizeof(int), st));
    if (N > 0) {
        map_tokens_kernel<<<grid_for(N, T256), T256, 0, st>>>(d_tokens, d_off, n, N, s->V, mtok, bad);
        int h_bad = 0;
        SD_CUDA_OK(cudaMemcpyAsync(&h_bad, bad, sizeof(int), cudaMemcpyDeviceToHost, st));
        SD_CUDA_OK(cudaStreamSynchronize(st));
        if (h_bad) return SD_ERR_INVALID_ARG;                    // nothing was changed yet
    }
    requests_prepare_kernel<<<(unsigned)n, T256, 0, st>>>(*s, n, d_slot, d_off, d_tokens);
    if (N > 0) {
        i64 max_len = 0;
        for (int q = 0; q < n; ++q) max_len = std::max<i64>(max_len, h_offsets[q + 1] - h_offsets[q]);
        // a handful of prompts: no round trips to the host on the way
        const bool small = N <= 65536;
        const int rc = pipeline_run(P, mtok, d_off, n, N, (i64)n * s->V, D, false, st, max_len, small);
        if (rc != SD_OK) return rc;
        requests_layout_kernel<<<grid_for(n, T256), T256, 0, st>>>(*s, n, d_off, P.nbase, P.runstart, P.lv.E, L);
        emit_nodes_slots_kernel<<<grid_for(N, T256), T256, 0, st>>>(*s, n, d_slot, d_off, mtok, P.sa, P.lcp, P.len, N, P.lv,
                                                                   P.nbase, P.nchild, P.runstart, L);
    } else {
        SD_CUDA_OK(cudaMemsetAsync(L.ok, 0xFF, sizeof(int) * n, st));
        SD_CUDA_OK(cudaMemsetAsync(L.used, 0, sizeof(int) * n, st));
        SD_CUDA_OK(cudaMemsetAsync(L.live, 0, sizeof(int) * n, st));
    }
    requests_finalize_kernel<<<grid_for((i64)n * 32, T256), T256, 0, st>>>(*s, n, d_slot, d_off, L);
    // (no synchronisation: the temporaries stay in the store's workspace, and a later call on
    // another stream must be ordered behind this one by the caller like any other use of the store)
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
