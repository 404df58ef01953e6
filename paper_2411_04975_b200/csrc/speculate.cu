// GenerateCandidateTree (Algorithm 1) for a whole batch.
//
// sd_speculate / sd_step: ONE launch, one thread block per request (speculate_fused_kernel):
//   - sd_step: warp 0 appends the request's accepted tokens to its tree (exactly what sd_append
//     does) while the other warps match and expand; only jobs through the request's tree wait;
//   - sd_step, blocks with many tokens to append: the other warps copy the request's text into
//     shared memory and scan it for the earlier occurrences of the last token: how many tokens before each one agree with the context says
//     which patterns it is an occurrence of.  A per-request match node with at most 32
//     occurrences needs no tree at all: a lane per occurrence, the node's sub-tree is read off
//     the text behind the occurrences (expand_occ).  Otherwise the per-request match nodes are
//     the slot's active nodes (sd_step: a job that needs them waits for the append);
//   - the global match nodes are advanced from the nodes cached at the previous call by
//     descending only the tokens appended since;
//   - the (tree, p) jobs go into a queue, costliest first, a warp per job; a job is dropped,
//     exactly, as soon as an upper bound of its SCORE falls below a score already reached;
//   - select (Section 3.2: only if SCORE > tau) and emit from shared memory.
// sd_speculate_noalloc: the two-kernel form, one warp per (request, tree, p) job with the jobs'
// records in global memory (match_expand_kernel, select_emit_kernel).
//
// fp64 rules: C = count / sibling-sum (Eq. 1), D = D(parent) * C (Eq. 2), SCORE
// adds D in insertion order; __ddiv_rn / __dmul_rn / __dadd_rn keep every
// operation a separately rounded IEEE binary64 operation (no FMA contraction).
#include <mutex>

#include "append_core.cuh"

namespace {

constexpr int SPEC_WARPS = 8;                 // warps per block of the job kernel
constexpr unsigned FULL = 0xffffffffu;

struct Frontier {                             // candidates of one job, best first, ring buffer
    double d[SD_MAX_SPEC];
    int tok[SD_MAX_SPEC];
    int par[SD_MAX_SPEC];
    int cb[SD_MAX_SPEC];
    unsigned nc[SD_MAX_SPEC];
};

// strict total order of candidates: larger D, then smaller token, then smaller parent index
// (D values are non-negative, so their bit patterns order like the values: branch-free compare.)
__device__ __forceinline__ bool better(double da, int ta, int pa, double db, int tb, int pb) {
    const long long a = __double_as_longlong(da), b = __double_as_longlong(db);
    return (a > b) | ((a == b) & ((ta < tb) | ((ta == tb) & (pa < pb))));
}

// Entry index of child `x` in the sorted run ent[cb .. cb+n), or -1.  Whole warp.
__device__ int find_child(const int4* __restrict__ ent, int cb, int n, int x, int lane) {
    int lo = 0, hi = n;
    for (int it = 0; it < 6 && hi - lo > 32; ++it) {       // window shrinks 33x per round
        const int q = lo + (int)(((long long)(hi - lo) * (lane + 1)) / 33);
        const int tk = ent[cb + q].x;
        const unsigned ge = __ballot_sync(FULL, tk >= x);
        const int f = ge ? __ffs(ge) - 1 : 32;              // first probe with token >= x
        const int q_prev = __shfl_sync(FULL, q, f > 0 ? f - 1 : 0);
        const int q_at = __shfl_sync(FULL, q, f < 32 ? f : 31);
        if (f > 0) lo = q_prev + 1;
        if (f < 32) hi = q_at + 1;
    }
    int found = -1;
    for (int base = lo; base < hi && found < 0; base += 32) {   // one round unless n is huge
        const int idx = base + lane;
        const bool hit = idx < hi && ent[cb + idx].x == x;
        const unsigned eq = __ballot_sync(FULL, hit);
        if (eq) found = cb + base + __ffs(eq) - 1;
    }
    return found;
}

// Insert one candidate (same values on every lane) into the sorted frontier of at
// most K entries.  fh = ring head, fs = size.
// Returns false if at least K entries are better (nothing changes then).
__device__ bool frontier_insert(Frontier& F, int fh, int& fs, int K, double d, int tok, int par, int cb, unsigned nc,
                                int lane) {
    const int i0 = lane, i1 = lane + 32;
    const int s0 = (fh + i0) & (SD_MAX_SPEC - 1), s1 = (fh + i1) & (SD_MAX_SPEC - 1);
    const bool b0 = i0 < fs && better(F.d[s0], F.tok[s0], F.par[s0], d, tok, par);
    const bool b1 = i1 < fs && better(F.d[s1], F.tok[s1], F.par[s1], d, tok, par);
    const int pos = __popc(__ballot_sync(FULL, b0)) + __popc(__ballot_sync(FULL, b1));
    if (pos >= K) return false;
    const int ns = min(fs + 1, K);
    double md0 = 0, md1 = 0; int mt0 = 0, mt1 = 0, mp0 = 0, mp1 = 0, mc0 = 0, mc1 = 0; unsigned mn0 = 0, mn1 = 0;
    const bool mv0 = i0 > pos && i0 < ns, mv1 = i1 > pos && i1 < ns;
    if (mv0) { const int q = (s0 - 1) & (SD_MAX_SPEC - 1); md0 = F.d[q]; mt0 = F.tok[q]; mp0 = F.par[q]; mc0 = F.cb[q]; mn0 = F.nc[q]; }
    if (mv1) { const int q = (s1 - 1) & (SD_MAX_SPEC - 1); md1 = F.d[q]; mt1 = F.tok[q]; mp1 = F.par[q]; mc1 = F.cb[q]; mn1 = F.nc[q]; }
    __syncwarp();
    if (mv0) { F.d[s0] = md0; F.tok[s0] = mt0; F.par[s0] = mp0; F.cb[s0] = mc0; F.nc[s0] = mn0; }
    if (mv1) { F.d[s1] = md1; F.tok[s1] = mt1; F.par[s1] = mp1; F.cb[s1] = mc1; F.nc[s1] = mn1; }
    if (i0 == pos) { F.d[s0] = d; F.tok[s0] = tok; F.par[s0] = par; F.cb[s0] = cb; F.nc[s0] = nc; }
    if (i1 == pos) { F.d[s1] = d; F.tok[s1] = tok; F.par[s1] = par; F.cb[s1] = cb; F.nc[s1] = nc; }
    __syncwarp();
    fs = ns;
    return true;
}

// Offer every child of a node (run ent[cb .. cb+n)) to the frontier.
__device__ void push_children(const int4* __restrict__ ent, int cb, int n, double d_parent, int par_index, Frontier& F,
                              int fh, int& fs, int K, int lane) {
    if (n <= 0 || K <= 0) return;
    long long sum = 0;
    int4 first = make_int4(0, 0, 0, 0);
    for (int base = 0; base < n; base += 32) {
        const int idx = base + lane;
        int4 e = make_int4(0, 0, 0, 0);
        if (idx < n) e = ent[cb + idx];
        if (base == 0) first = e;
        sum += e.y;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
    const double dsum = (double)sum;                            // denominator of Eq. 1
    for (int base = 0; base < n; base += 32) {
        const int idx = base + lane;
        const bool v = idx < n;
        int4 e = first;
        if (base != 0) { e = make_int4(0, 0, 0, 0); if (v) e = ent[cb + idx]; }
        double dc = 0.0;
        if (v) dc = __dmul_rn(d_parent, __ddiv_rn((double)e.y, dsum));   // Eq. 2 with Eq. 1
        bool pass = v;
        if (v && fs == K) {                                     // cannot beat the current worst: skip
            const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
            pass = better(dc, e.x, par_index, F.d[last], F.tok[last], F.par[last]);
        }
        unsigned m = __ballot_sync(FULL, pass);
        while (m) {
            const int src = __ffs(m) - 1;
            m &= m - 1;
            const double cd = __shfl_sync(FULL, dc, src);
            const int ct = __shfl_sync(FULL, e.x, src);
            const int cc = __shfl_sync(FULL, e.z, src);
            const unsigned cn = (unsigned)__shfl_sync(FULL, e.w, src);
            frontier_insert(F, fh, fs, K, cd, ct, par_index, cc, cn, lane);
        }
    }
}

__device__ __forceinline__ int budget_for(double alpha, int p, int cap) {
    const double b = floor(__dmul_rn(alpha, (double)p));        // Eq. 3
    if (b > (double)cap) return cap;
    if (b < 0.0) return 0;
    return (int)b;
}

__global__ void __launch_bounds__(SPEC_WARPS * 32)
match_expand_kernel(sd_store sv, int n, const int32_t* __restrict__ d_slot, int Pe, double alpha, int max_spec,
                    unsigned flags, const int32_t* __restrict__ d_budget_cap) {
    __shared__ Frontier fr[SPEC_WARPS];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const long long job = (long long)blockIdx.x * SPEC_WARPS + wib;
    if (job >= (long long)n * 2 * Pe) return;
    const int i = (int)(job / (2 * Pe));
    const int rem = (int)(job % (2 * Pe));
    const int tree = rem / Pe, p = rem % Pe + 1;
    const long long rec = ((long long)i * 2 + tree) * sv.D + (p - 1);
    int cnt = 0;
    double score = 0.0;
    const int slot = d_slot[i];
    bool live = slot >= 0 && slot < sv.R;
    if (tree == 0 && (flags & SD_FLAG_REQUEST_ONLY)) live = false;
    if (tree == 1 && (flags & SD_FLAG_GLOBAL_ONLY)) live = false;
    if (live) {
        const SlotState* ss = sv.s_state + slot;
        const int t = ss->len;
        if (ss->status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN)) live = false;
        if (p > t) live = false;
        int cap = max_spec;
        if (d_budget_cap && d_budget_cap[i] >= 0) cap = min(cap, d_budget_cap[i]);
        const int budget = budget_for(alpha, p, cap);
        if (live && budget > 0) {
            // ---- MatchPattern
            const int4* ent;
            int node;
            if (tree == 1) {
                ent = sv.s_ent + (long long)slot * sv.spn;
                node = ss->active[p - 1];                       // node of the last p tokens
            } else {
                ent = sv.g_ent;
                const int32_t* pat = sv.s_text + (long long)slot * sv.T + (t - p);
                node = sv.g_root[pat[0]];
                for (int k = 1; k < p && node >= 0; ++k) {
                    const int4 e = ent[node];
                    node = find_child(ent, e.z, (int)((unsigned)e.w & RUN_COUNT_MASK), pat[k], lane);
                }
            }
            if (node >= 0) {
                // ---- ExpandSpeculationTree
                Frontier& F = fr[wib];
                int fh = 0, fs = 0;
                const int4 e = ent[node];
                push_children(ent, e.z, (int)((unsigned)e.w & RUN_COUNT_MASK), 1.0, -1, F, fh, fs, budget, lane);
                int32_t* out_tok = sv.j_tok + rec * sv.M;
                int32_t* out_par = sv.j_par + rec * sv.M;
                while (cnt < budget && fs > 0) {
                    const double d = F.d[fh];
                    const int tok = F.tok[fh], par = F.par[fh], cb = F.cb[fh];
                    const int nc = (int)(F.nc[fh] & RUN_COUNT_MASK);
                    __syncwarp();
                    fh = (fh + 1) & (SD_MAX_SPEC - 1);
                    --fs;
                    if (lane == 0) { out_tok[cnt] = tok; out_par[cnt] = par; }
                    score = __dadd_rn(score, d);                // Eq. 4, insertion order
                    const int idx = cnt++;
                    const int K = budget - cnt;
                    if (fs > K) fs = K;
                    if (flags & SD_FLAG_LINEAR) fs = 0;
                    push_children(ent, cb, nc, d, idx, F, fh, fs, K, lane);
                }
            }
        }
    }
    if (lane == 0) { sv.j_n[rec] = cnt; sv.j_score[rec] = score; }
}

__global__ void select_emit_kernel(sd_store sv, int n, const int32_t* __restrict__ d_slot, int Pe, double tau, int32_t* d_n_draft,
                                   int32_t* d_tokens, int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask,
                                   int32_t* d_chosen_tree, int32_t* d_chosen_p, double* d_score, int32_t* d_status) {
    __shared__ int spar[4][SD_MAX_SPEC];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int i = blockIdx.x * 4 + wib;
    if (i >= n) return;
    const int M = sv.M, words = (M + 31) / 32;
    const int slot = d_slot[i];
    const bool ok = slot >= 0 && slot < sv.R;
    // first job in loop order (global before per-request, p ascending) with the largest score
    double best = 0.0;
    int best_o = -1;
    for (int o = lane; o < 2 * Pe; o += 32) {
        const long long rec = ((long long)i * 2 + o / Pe) * sv.D + (o % Pe);
        const double sc = sv.j_score[rec];
        if (sc > best) { best = sc; best_o = o; }               // ascending o: strict '>' keeps the first
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const double ob = __shfl_xor_sync(FULL, best, off);
        const int oo = __shfl_xor_sync(FULL, best_o, off);
        if (oo >= 0 && (ob > best || (ob == best && (best_o < 0 || oo < best_o)))) { best = ob; best_o = oo; }
    }
    int nd = 0, tree = -1, p = 0, t = 0, status = SD_STATUS_BAD_SLOT;
    long long rec = 0;
    if (ok) {
        t = sv.s_state[slot].len;
        status = sv.s_state[slot].status;
    }
    if (ok && best_o >= 0 && best > tau) {                      // Section 3.2: only a score above the threshold is used
        tree = best_o / Pe; p = best_o % Pe + 1;
        rec = ((long long)i * 2 + tree) * sv.D + (p - 1);
        nd = sv.j_n[rec];
    } else {
        best = 0.0;
    }
    for (int j = lane; j < SD_MAX_SPEC; j += 32) spar[wib][j] = j < nd ? sv.j_par[rec * M + j] : -1;
    __syncwarp();
    for (int j = lane; j < M; j += 32) {
        int tok = -1, par = -1, pos = -1;
        unsigned long long bits = 0;
        if (j < nd) {
            tok = sv.j_tok[rec * M + j];
            par = spar[wib][j];
            int depth = 0;
            for (int a = j, hops = 0; a >= 0 && hops < SD_MAX_SPEC; a = spar[wib][a], ++hops) {
                bits |= 1ull << a;
                ++depth;
            }
            pos = t + depth - 1;
        }
        const long long o = (long long)i * M + j;
        d_tokens[o] = tok; d_parents[o] = par; d_positions[o] = pos;
        d_mask[o * words] = (uint32_t)bits;
        if (words > 1) d_mask[o * words + 1] = (uint32_t)(bits >> 32);
    }
    if (lane == 0) {
        d_n_draft[i] = nd; d_chosen_tree[i] = tree; d_chosen_p[i] = p; d_score[i] = best;
        if (d_status) d_status[i] = status;
    }
}


// ---------------------------------------------------------------------------------------------
// Fused path: one block of W warps per request (the kernel itself is described where it is
// defined).  Two blocks per SM is the usual shape: W = 10 with 96 registers per thread.  A batch
// of at most one request per SM gets bigger blocks (W = 24 / 16), a batch of more than two
// requests per SM smaller ones (W = 8 / 5, four per SM) to stay in one wave.
constexpr int CTA_WARPS = 10;                  // the usual block (96 registers; 16 warps x 64 registers spill: 87 us against 83.5)
constexpr int CTA_WARPS_STEP = 10;             // the usual block of sd_step: 10 warps with 96 registers each and
constexpr int STEP_G = 4;                      // an append that moves four entries per round, so that the
                                               // append in front does not spill.  Measured per step: 92.7 us;
                                               // 9 warps 92.8, 11 (80 registers) 95, 8 (128) 96; with eight
                                               // entries per round: 8 warps x 128 registers 95, 10 x 96 100,
                                               // 12 x 80 100, 16 x 64 104, 6 x 168 110
constexpr int CTA_WARPS_WIDE = 24;             // small batches (one block per SM at most): the block has the SM's
constexpr int CTA_WARPS_WIDE_STEP = 16;        // registers to itself (80 per thread; sd_step: 128)
constexpr int CTA_WARPS_NARROW = 8;            // batches of more than two requests per SM: four blocks per SM
constexpr int CTA_WARPS_NARROW_STEP = 5;       // (sd_step: 96 registers and the four-entry append; 512 requests:
                                               // 82 us per step, 88 with 4 warps x 128 registers, 100 with 8 x 64)

struct WarpWork {
    Frontier F;
    Frontier T;                               // scratch list for the children of one wide node
    int one_tok[SD_MAX_SPEC];                 // its first children of count 1, in token order
    int one_cb[SD_MAX_SPEC];
    unsigned one_nc[SD_MAX_SPEC];
    int tok[2][SD_MAX_SPEC];                  // draft tokens: working buffer and best-so-far buffer
    unsigned char par[2][SD_MAX_SPEC];        // parent index + 1 (0: child of the match node)
    double best_score;
    int best_order, best_n, best_buf;
};

template <int WARPS>
struct BlockSharedT {
    WarpWork w[WARPS];
    int node[2][SD_MAX_DEPTH];                // match node per tree and pattern length (-1: none)
    int cb[2][SD_MAX_DEPTH];                  // its child run
    unsigned nc[2][SD_MAX_DEPTH];             // ... as the node's w field (count | flags)
    int cost[2 * SD_MAX_DEPTH];
    int job[2 * SD_MAX_DEPTH];
    int wide[2 * SD_MAX_DEPTH];               // jobs whose match node has a wide child run
    int njobs, next, nwide, nwide_kept;
    long long slice_sum[WARPS];
    int slice_fs[WARPS];
    // per-request tree, read off the text: earlier occurrences of the last token by the number of
    // tokens before them that agree with the context
    int r_hist[SD_MAX_DEPTH + 2];
    int r_cum[SD_MAX_DEPTH + 2];              // r_cum[p]: occurrences of the pattern of length p
    int r_fill[SD_MAX_DEPTH + 2];
    int r_list[SD_OCC_LANES];                 // the occurrences of the patterns that have at most 32, longest matches first
    int r_pn;                                 // shortest such pattern
    int app_done;                             // sd_step: warp 0 has appended the new tokens
    int nlate, late[SD_MAX_DEPTH];            // per-request jobs whose wait for the append ran out
    int scan_next[2];
    unsigned best_hi;                         // high word of the largest SCORE reached so far: a lower
                                              // bound of it (scores are non-negative doubles), which is
                                              // all the pruning needs; 32 bits keep the atomic native
    int win_warp;
};

// find_child that also hands back the matched entry (valid when the result is >= 0)
__device__ int find_child_entry(const int4* __restrict__ ent, int cb, int n, int x, int lane, int4& out) {
    int lo = 0, hi = n;
    for (int it = 0; it < 6 && hi - lo > 32; ++it) {
        const int q = lo + (int)(((long long)(hi - lo) * (lane + 1)) / 33);
        const int tk = ent[cb + q].x;
        const unsigned ge = __ballot_sync(FULL, tk >= x);
        const int f = ge ? __ffs(ge) - 1 : 32;
        const int q_prev = __shfl_sync(FULL, q, f > 0 ? f - 1 : 0);
        const int q_at = __shfl_sync(FULL, q, f < 32 ? f : 31);
        if (f > 0) lo = q_prev + 1;
        if (f < 32) hi = q_at + 1;
    }
    int found = -1;
    for (int base = lo; base < hi && found < 0; base += 32) {
        const int idx = base + lane;
        int4 e = make_int4(-1, 0, 0, 0);
        if (idx < hi) e = ent[cb + idx];
        const unsigned eq = __ballot_sync(FULL, idx < hi && e.x == x);
        if (eq) {
            const int src = __ffs(eq) - 1;
            found = cb + base + src;
            out.x = __shfl_sync(FULL, e.x, src); out.y = __shfl_sync(FULL, e.y, src);
            out.z = __shfl_sync(FULL, e.z, src); out.w = __shfl_sync(FULL, e.w, src);
        }
    }
    return found;
}



__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// Start fetching the `n` entries at ent[cb ...] into L2 (whole warp; at most `max_lines` 128-byte lines per lane).
__device__ __forceinline__ void prefetch_run(const int4* __restrict__ ent, int cb, int n, int lane, int max_rounds) {
    const int lines = (n + 7) >> 3;
    for (int r = 0, l = lane; r < max_rounds && l < lines; ++r, l += 32) prefetch_l2(ent + cb + l * 8);
}

// Merge up to 32 candidates (one per lane with `pass`) into the sorted frontier of at most K
// entries in one go: every survivor's final position is its number of betters, found by
// broadcasting the candidates once; then all entries move together.
__device__ void frontier_merge(Frontier& F, int fh, int& fs, int K, bool pass, double d, int tok, int par, int cb,
                               unsigned nc, int lane) {
    const unsigned m = __ballot_sync(FULL, pass);
    if (!m) return;
    const int i0 = lane, i1 = lane + 32;
    const int s0 = (fh + i0) & (SD_MAX_SPEC - 1), s1 = (fh + i1) & (SD_MAX_SPEC - 1);
    const bool v0 = i0 < fs, v1 = i1 < fs;
    double e0d = 0.0, e1d = 0.0;
    int e0t = 0, e1t = 0, e0p = 0, e1p = 0;
    if (v0) { e0d = F.d[s0]; e0t = F.tok[s0]; e0p = F.par[s0]; }
    if (v1) { e1d = F.d[s1]; e1t = F.tok[s1]; e1p = F.par[s1]; }
    int up0 = 0, up1 = 0;                                       // candidates that go before E[i0], E[i1]
    int my_rank = 0;
    unsigned mm = m;
    while (mm) {
        const int src = __ffs(mm) - 1;
        mm &= mm - 1;
        const double bd = __shfl_sync(FULL, d, src);
        const int bt = __shfl_sync(FULL, tok, src), bp = __shfl_sync(FULL, par, src);
        const bool b0 = v0 && better(bd, bt, bp, e0d, e0t, e0p);
        const bool b1 = v1 && better(bd, bt, bp, e1d, e1t, e1p);
        up0 += b0 ? 1 : 0;
        up1 += b1 ? 1 : 0;
        const int worse_old = __popc(__ballot_sync(FULL, b0)) + __popc(__ballot_sync(FULL, b1));
        const int better_new = __popc(__ballot_sync(FULL, pass && lane != src && better(d, tok, par, bd, bt, bp)));
        if (lane == src) my_rank = (fs - worse_old) + better_new;
    }
    const int n0 = i0 + up0, n1 = i1 + up1;
    int c0 = 0, c1 = 0;
    unsigned w0 = 0, w1 = 0;
    const bool k0 = v0 && n0 < K && up0 > 0, k1 = v1 && n1 < K && up1 > 0;   // entries that move
    if (k0) { c0 = F.cb[s0]; w0 = F.nc[s0]; }
    if (k1) { c1 = F.cb[s1]; w1 = F.nc[s1]; }
    __syncwarp();
    if (k0) { const int q = (fh + n0) & (SD_MAX_SPEC - 1); F.d[q] = e0d; F.tok[q] = e0t; F.par[q] = e0p; F.cb[q] = c0; F.nc[q] = w0; }
    if (k1) { const int q = (fh + n1) & (SD_MAX_SPEC - 1); F.d[q] = e1d; F.tok[q] = e1t; F.par[q] = e1p; F.cb[q] = c1; F.nc[q] = w1; }
    if (pass && my_rank < K) {
        const int q = (fh + my_rank) & (SD_MAX_SPEC - 1);
        F.d[q] = d; F.tok[q] = tok; F.par[q] = par; F.cb[q] = cb; F.nc[q] = nc;
    }
    __syncwarp();
    fs = min(fs + __popc(m), K);
}

// Offer the first `cnt` entries of list O (ordered, ring head 0) to F.
__device__ void frontier_merge_list(Frontier& F, int fh, int& fs, int K, const Frontier& O, int cnt, int par, int lane) {
    for (int base = 0; base < cnt; base += 32) {
        const int q = base + lane;
        bool pass = q < cnt;
        double d = 0.0; int tok = 0, cb = 0; unsigned nc = 0;
        if (pass) { d = O.d[q]; tok = O.tok[q]; cb = O.cb[q]; nc = O.nc[q]; }
        if (pass && fs == K) {
            const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
            pass = better(d, tok, par, F.d[last], F.tok[last], F.par[last]);
        }
        if (!__any_sync(FULL, pass)) break;                     // O is ordered: nothing further can enter
        frontier_merge(F, fh, fs, K, pass, d, tok, par, cb, nc, lane);
    }
}

// A WINDOW is 32 consecutive entries, one per lane, starting at `base`.  Trees are laid out so
// that the child run of a node's first (often only) child tends to follow the node's own
// child run, so one window usually holds several levels of a path at once.
__device__ __forceinline__ int4 load_window(const int4* __restrict__ ent, int base, int limit, int lane) {
    const int idx = base + lane;
    // the entries behind the window hold the rest of the node's sub-tree (pre-order layout):
    // bring the next 1.5 KB into L2 so that the following windows of this job hit there
    if (lane < 12 && base + 32 + lane * 8 < limit)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(ent + base + 32 + lane * 8));
    return idx < limit ? ent[idx] : make_int4(-1, 0, 0, 0);
}

// A child that was not put into the frontier because it would be taken out again at once.
struct Taken {
    bool any;
    double d;
    int tok, cb;
    unsigned w;
};

// Offer the children of a node to the frontier; `w` already holds the first 32 entries of the run.
// With `take` (runs of at most 32 children): if the best child (largest count, then smallest
// token: among siblings that is the order of D) beats every waiting candidate, it is the next
// node to be added whatever else is offered, so it is handed back instead of being merged in
// and popped again; the frontier is then bounded by K - 1.
__device__ void push_children_w(const int4* __restrict__ ent, int cb, int n, int4 w, double d_parent, int par_index,
                                Frontier& F, int fh, int& fs, int K, int lane, Taken* take = nullptr) {
    if (take) take->any = false;
    if (n <= 0 || K <= 0) return;
    // sibling sum: the denominator of Eq. 1 (a parent's occurrences fit 31 bits)
    unsigned part = lane < n ? (unsigned)w.y : 0u;
    for (int base = 32; base < n; base += 128) {                // wide runs: four loads in flight
        int y[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { const int idx = base + u * 32 + lane; y[u] = idx < n ? ent[cb + idx].y : 0; }
        part += (unsigned)(y[0] + y[1] + y[2] + y[3]);
    }
    const unsigned sum = __reduce_add_sync(FULL, part);
    const double dsum = (double)sum;
    int skip = -1;                                              // child handed back through `take`
    if (take && n <= 32) {
        const unsigned cmax = __reduce_max_sync(FULL, lane < n ? (unsigned)w.y : 0u);
        const int b = __ffs(__ballot_sync(FULL, lane < n && (unsigned)w.y == cmax)) - 1;
        const double db = __dmul_rn(d_parent, __ddiv_rn((double)cmax, dsum));    // Eq. 2 with Eq. 1
        const int tb = __shfl_sync(FULL, w.x, b);
        if (fs == 0 || better(db, tb, par_index, F.d[fh], F.tok[fh], F.par[fh])) {
            take->any = true; take->d = db; take->tok = tb;
            take->cb = __shfl_sync(FULL, w.z, b);
            take->w = (unsigned)__shfl_sync(FULL, w.w, b);
            skip = b;
            --K;                                                // one node fewer is still to come
            if (fs > K) fs = K;
            if (K <= 0 || n == 1) return;
        }
    }
    // With a full frontier only a child that beats its worst entry matters:
    // D = d_parent * count / sum, so counts below `cmin` lose without any fp64 work.
    double ld = 0.0, need = 0.0; int lt = 0, lp = 0;
    const bool full = fs == K;
    if (full) {
        const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
        ld = F.d[last]; lt = F.tok[last]; lp = F.par[last];
        need = ld * dsum * 0.999999;                            // count * d_parent must reach this
    }
    for (int base = 0; base < n; base += 32) {
        const int idx = base + lane;
        int4 e = w;
        if (base != 0) { e = make_int4(0, 0, 0, 0); if (idx < n) e = ent[cb + idx]; }
        bool pass = idx < n && idx != skip && (double)e.y * d_parent >= need;
        if (!__any_sync(FULL, pass)) continue;
        double dc = 0.0;
        if (pass) {
            dc = __dmul_rn(d_parent, __ddiv_rn((double)e.y, dsum));      // Eq. 2 with Eq. 1
            if (full) pass = better(dc, e.x, par_index, ld, lt, lp);
            if (pass && ((unsigned)e.w & RUN_COUNT_MASK)) prefetch_l2(ent + e.z);   // likely looked at soon
        }
        if (fs == 0 && n <= 32) {
            // Nothing waits yet (the first children of a job): the candidates are siblings, and
            // among siblings the order of D is the order of (count, then token).  Their places
            // follow from one pass per distinct count, largest first, without any merging.
            unsigned rem = __ballot_sync(FULL, pass);
            const int np = __popc(rem);
            const unsigned below = (1u << lane) - 1u;
            int place = -1, taken = 0;
            while (rem && taken < K) {
                const bool in = (rem >> lane) & 1u;
                const unsigned top = __reduce_max_sync(FULL, in ? (unsigned)e.y : 0u);
                const unsigned grp = __ballot_sync(FULL, in && (unsigned)e.y == top);
                if ((grp >> lane) & 1u) place = taken + __popc(grp & below);
                taken += __popc(grp);
                rem &= ~grp;
            }
            if (place >= 0 && place < K) {
                const int q = (fh + place) & (SD_MAX_SPEC - 1);
                F.d[q] = dc; F.tok[q] = e.x; F.par[q] = par_index; F.cb[q] = e.z; F.nc[q] = (unsigned)e.w;
            }
            __syncwarp();
            fs = min(np, K);
            return;
        }
        frontier_merge(F, fh, fs, K, pass, dc, e.x, par_index, e.z, (unsigned)e.w, lane);
        if (!full && fs == K) {                                 // it filled up while merging
            const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
            const double d2 = F.d[last];
            const int t2 = F.tok[last], p2 = F.par[last];
            // from here on compare exactly against the new worst entry (no count shortcut)
            for (int b2 = base + 32; b2 < n; b2 += 32) {
                const int i2 = b2 + lane;
                int4 e2 = make_int4(0, 0, 0, 0);
                if (i2 < n) e2 = ent[cb + i2];
                double dc2 = 0.0;
                bool pass2 = i2 < n;
                if (pass2) {
                    dc2 = __dmul_rn(d_parent, __ddiv_rn((double)e2.y, dsum));
                    const int l3 = (fh + fs - 1) & (SD_MAX_SPEC - 1);
                    pass2 = better(dc2, e2.x, par_index, F.d[l3], F.tok[l3], F.par[l3]);
                }
                frontier_merge(F, fh, fs, K, pass2, dc2, e2.x, par_index, e2.z, (unsigned)e2.w, lane);
            }
            (void)d2; (void)t2; (void)p2;
            return;
        }
    }
}

// MatchPattern from a known node: descend text[from .. to).  Levels whose child run lies inside
// the window already in registers cost no memory access.  Returns the node reached (-1: no
// match) and its child run in (cb, n).
// The context is `text` up to position t_old and `newtok` from there on (tokens that are
// being appended in the same launch).
__device__ int walk_from(const int4* __restrict__ ent, int limit, int node, const int32_t* __restrict__ text, int t_old,
                         const int32_t* __restrict__ newtok, int from, int to, int lane, int& cb, unsigned& wfull) {
    if (node < 0) return -1;
    int wb = node;
    int4 w = load_window(ent, wb, limit, lane);
    cb = __shfl_sync(FULL, w.z, 0);
    wfull = (unsigned)__shfl_sync(FULL, w.w, 0);
    int n = (int)(wfull & RUN_COUNT_MASK);
    for (int pos = from; pos < to; ++pos) {
        const int x = pos < t_old ? text[pos] : newtok[pos - t_old];
        if (n == 0) return -1;
        if (n > 32) {                                           // wide run: 32-way search
            int4 e;
            node = find_child_entry(ent, cb, n, x, lane, e);
            if (node < 0) return -1;
            cb = e.z; wfull = (unsigned)e.w; n = (int)(wfull & RUN_COUNT_MASK);
            wb = -64;                                           // no usable window
            continue;
        }
        if (!(cb >= wb && cb + n <= wb + 32)) { wb = cb; w = load_window(ent, wb, limit, lane); }
        const int rel = wb + lane - cb;
        const unsigned hit = __ballot_sync(FULL, rel >= 0 && rel < n && w.x == x);
        if (!hit) return -1;
        const int src = __ffs(hit) - 1;
        node = wb + src;
        cb = __shfl_sync(FULL, w.z, src);
        wfull = (unsigned)__shfl_sync(FULL, w.w, src);
        n = (int)(wfull & RUN_COUNT_MASK);
    }
    return node;
}


// Children of a node whose run has a top block (see RUN_HAS_TOP): the 64 best by count are
// listed, best first, right before the run, together with the sum of all counts.
__device__ void push_top(const int4* __restrict__ ent, int cb, double d_parent, int par_index, Frontier& F, int fh,
                         int& fs, int K, int lane) {
    if (K <= 0) return;
    const int4 hdr = ent[cb - SD_TOP_BLOCK];
    const double dsum = (double)(((unsigned long long)(unsigned)hdr.y << 32) | (unsigned long long)(unsigned)hdr.x);
    const int ntop = min(hdr.z, K);                             // only the K best can enter
    for (int base = 0; base < ntop; base += 32) {
        const int idx = base + lane;
        bool pass = idx < ntop;
        int4 e = make_int4(0, 0, 0, 0);
        double dc = 0.0;
        if (pass) {
            e = ent[cb - SD_TOP_BLOCK + 1 + idx];
            dc = __dmul_rn(d_parent, __ddiv_rn((double)e.y, dsum));      // Eq. 2 with Eq. 1
            if (fs == K) {
                const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
                pass = better(dc, e.x, par_index, F.d[last], F.tok[last], F.par[last]);
            }
            if (pass && ((unsigned)e.w & RUN_COUNT_MASK)) prefetch_l2(ent + e.z);
        }
        if (!__any_sync(FULL, pass)) break;                     // best first: nothing further can enter
        frontier_merge(F, fh, fs, K, pass, dc, e.x, par_index, e.z, (unsigned)e.w, lane);
    }
}

constexpr int WIDE_RUN = 256;                 // child runs longer than this are scanned by several warps

// One pass over chunks first, first + stride, ... of a child run: adds up the counts and keeps
// the K children with the largest counts (then smallest tokens) in F, ordered, with the COUNT
// in the d field.  Among the children of one parent that is the order of D (Eq. 2), so no
// division is needed while scanning.  F starts empty at ring head fh.
// Most children of a wide node occur once.  Those tie on the count and rank by token, i.e. in
// run order: the first K of them are simply copied (ones list) and appended behind the
// children that occur more often, which alone go through the ordered merge.
// Children with a count below `cmin` are known not to matter and are skipped.
__device__ void scan_run_by_count(const int4* __restrict__ ent, int cb, int n, int first, int stride, int par_index,
                                  int cmin, WarpWork& W, Frontier& F, int fh, int& fs, int K, long long& sum_out,
                                  int lane) {
    long long sum = 0;
    fs = 0;
    int ones = 0;                                               // count-1 children copied so far (warp-uniform)
    if (stride == 1) prefetch_run(ent, cb, n, lane, 64);        // the whole run, all lines in flight at once
    for (int c = first; c * 32 < n; c += 4 * stride) {
        int4 e[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {                           // four loads in flight
            const int idx = (c + u * stride) * 32 + lane;
            e[u] = make_int4(-1, 0, 0, 0);
            if (idx < n) e[u] = ent[cb + idx];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            sum += e[u].y;
            const unsigned m1 = __ballot_sync(FULL, e[u].y == 1 && cmin <= 1);
            if (m1 && ones < K) {
                const int at = ones + __popc(m1 & ((1u << lane) - 1u));
                if (e[u].y == 1 && at < K) { W.one_tok[at] = e[u].x; W.one_cb[at] = e[u].z; W.one_nc[at] = (unsigned)e[u].w; }
                ones = min(K, ones + __popc(m1));
            }
            bool pass = e[u].y >= 2 && e[u].y >= cmin;
            if (pass && fs == K) {
                const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
                pass = better((double)e[u].y, e[u].x, par_index, F.d[last], F.tok[last], F.par[last]);
            }
            if (pass && ((unsigned)e[u].w & RUN_COUNT_MASK)) prefetch_l2(ent + e[u].z);
            frontier_merge(F, fh, fs, K, pass, (double)e[u].y, e[u].x, par_index, e[u].z, (unsigned)e[u].w, lane);
        }
    }
    __syncwarp();
    // the count-1 children go behind the others, in token order, as far as there is room
    const int take = min(ones, K - fs);
    for (int i = lane; i < take; i += 32) {
        const int q = (fh + fs + i) & (SD_MAX_SPEC - 1);
        F.d[q] = 1.0; F.tok[q] = W.one_tok[i]; F.par[q] = par_index; F.cb[q] = W.one_cb[i]; F.nc[q] = W.one_nc[i];
    }
    fs += take;
    __syncwarp();
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
    sum_out = sum;
}

// counts in F.d -> D = d_parent * count / sum (Eq. 1, Eq. 2)
__device__ void counts_to_d(Frontier& F, int fh, int fs, double d_parent, long long sum, int lane) {
    const double dsum = (double)sum;
    for (int i = lane; i < fs; i += 32) {
        const int q = (fh + i) & (SD_MAX_SPEC - 1);
        F.d[q] = __dmul_rn(d_parent, __ddiv_rn(F.d[q], dsum));
    }
    __syncwarp();
}

template <class BlockShared>
__device__ __forceinline__ double best_so_far(BlockShared& sh) {
    return __hiloint2double((int)__shfl_sync(FULL, *(volatile unsigned*)&sh.best_hi, 0), 0);
}

// ExpandSpeculationTree + SCORE for one (tree, p) job by one warp.  With `seeded` the frontier
// already holds the match node's children (fs entries from ring head 0).
template <class BlockShared>
__device__ void expand_job(BlockShared& sh, WarpWork& W, const int4* __restrict__ ent, int limit, int tree, int p,
                           int budget, unsigned flags, bool seeded, int fs, int lane) {
    const int order = tree * SD_MAX_DEPTH + p;                  // loop order of Algorithm 1
    const int buf = W.best_buf ^ 1;
    int fh = 0, cnt = 0;
    double score = 0.0;
    bool dropped = false;
    // the node whose children are to be offered next: the match node first, D(N_p) = 1
    double cur_d = 1.0;
    int cur_cb = sh.cb[tree][p - 1], cur_idx = -1;
    unsigned cur_w = sh.nc[tree][p - 1];
    int cur_n = (int)(cur_w & RUN_COUNT_MASK);
    bool have_cur = !seeded;
    if (!seeded) fs = 0;
    int4 w = make_int4(-1, 0, 0, 0);                            // window in registers: entries wb .. wb + wvalid
    int wb = -1, wvalid = 0;
    while (true) {
        if (!have_cur) {
            if (cnt >= budget || fs == 0) break;
            cur_d = W.F.d[fh];
            const int tok = W.F.tok[fh], par = W.F.par[fh];
            cur_cb = W.F.cb[fh];
            cur_w = W.F.nc[fh];
            cur_n = (int)(cur_w & RUN_COUNT_MASK);
            // everything still to come is at most cur_d each
            if ((score + (double)(budget - cnt) * cur_d) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
            __syncwarp();
            fh = (fh + 1) & (SD_MAX_SPEC - 1);
            --fs;
            if (lane == 0) { W.tok[buf][cnt] = tok; W.par[buf][cnt] = (unsigned char)(par + 1); }
            score = __dadd_rn(score, cur_d);                    // Eq. 4, insertion order
            // the final SCORE of this job is at least its running value: let the others prune on it
            if (lane == 0) atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
            cur_idx = cnt++;
            const int K = budget - cnt;
            if (fs > K) fs = K;
            if (flags & SD_FLAG_LINEAR) fs = 0;
        }
        have_cur = false;
        if (cnt >= budget) break;
        if (cur_n == 0) continue;
        if (cur_w & RUN_HAS_TOP) {                              // long run with a ready-made list of its best children
            push_top(ent, cur_cb, cur_d, cur_idx, W.F, fh, fs, budget - cnt, lane);
            continue;
        }
        if (cur_n > 32) {
            // wide run: one pass that keeps the best children by count, then D for those only
            const int K = budget - cnt;
            long long sum;
            if (fs == 0) {
                scan_run_by_count(ent, cur_cb, cur_n, 0, 1, cur_idx, 1, W, W.F, fh, fs, K, sum, lane);
                counts_to_d(W.F, fh, fs, cur_d, sum, lane);
            } else if (fs == K) {
                // full frontier: sum pass, then a pass that only looks at counts large enough
                prefetch_run(ent, cur_cb, cur_n, lane, 64);
                push_children_w(ent, cur_cb, cur_n, load_window(ent, cur_cb, limit, lane), cur_d, cur_idx, W.F, fh, fs, K,
                                lane);
            } else {
                // some candidates wait and there is room for more: the K best children by count go
                // into a list of their own, which is then merged in
                int ts;
                scan_run_by_count(ent, cur_cb, cur_n, 0, 1, cur_idx, 1, W, W.T, 0, ts, K, sum, lane);
                counts_to_d(W.T, 0, ts, cur_d, sum, lane);
                frontier_merge_list(W.F, fh, fs, K, W.T, ts, cur_idx, lane);
            }
            continue;
        }
        {
            const int off = cur_cb - wb;
            if (wb >= 0 && off >= 0 && off + cur_n <= wvalid) {  // the run is already in registers
                if (off > 0) {
                    w.x = __shfl_down_sync(FULL, w.x, off); w.y = __shfl_down_sync(FULL, w.y, off);
                    w.z = __shfl_down_sync(FULL, w.z, off); w.w = __shfl_down_sync(FULL, w.w, off);
                    wvalid -= off;
                    wb = cur_cb;
                }
            } else {
                w = load_window(ent, cur_cb, limit, lane);
                wb = cur_cb;
                wvalid = min(32, limit - cur_cb);
            }
        }
        if (cur_n == 1 && (fs == 0 || W.F.d[fh] < cur_d)) {
            // An only child has C = 1, so D stays cur_d: while the best waiting candidate is
            // strictly worse, the whole chain of only children is added in one go.
            const bool link = lane < wvalid && ((unsigned)w.w & RUN_COUNT_MASK) == 1u && w.z == cur_cb + lane + 1;
            const unsigned links = __ballot_sync(FULL, link);
            const int len = min(wvalid, 1 + (links == 0xffffffffu ? 32 : __ffs(~links) - 1));
            const int m = min(len, budget - cnt);
            if (lane < m) {
                W.tok[buf][cnt + lane] = w.x;
                W.par[buf][cnt + lane] = (unsigned char)((lane == 0 ? cur_idx : cnt + lane - 1) + 1);
            }
            for (int q = 0; q < m; ++q) score = __dadd_rn(score, cur_d);
            if (lane == 0) atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
            cnt += m;
            if (fs > budget - cnt) fs = budget - cnt;
            cur_idx = cnt - 1;
            cur_cb = __shfl_sync(FULL, w.z, m - 1);
            cur_w = (unsigned)__shfl_sync(FULL, w.w, m - 1);
            cur_n = (int)(cur_w & RUN_COUNT_MASK);
            have_cur = true;
            if ((score + (double)(budget - cnt) * cur_d) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
            continue;
        }
        Taken tk;
        push_children_w(ent, cur_cb, cur_n, w, cur_d, cur_idx, W.F, fh, fs, budget - cnt, lane, &tk);
        if (tk.any) {
            // the same steps as taking it from the frontier at the top of the loop
            if ((score + (double)(budget - cnt) * tk.d) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
            if (lane == 0) { W.tok[buf][cnt] = tk.tok; W.par[buf][cnt] = (unsigned char)(cur_idx + 1); }
            score = __dadd_rn(score, tk.d);
            if (lane == 0) atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
            cur_idx = cnt++;
            cur_d = tk.d; cur_cb = tk.cb; cur_w = tk.w;
            cur_n = (int)(cur_w & RUN_COUNT_MASK);
            if (flags & SD_FLAG_LINEAR) fs = 0;
            have_cur = true;
        }
    }
    __syncwarp();
    if (!dropped && (score > W.best_score || (score == W.best_score && score > 0.0 && order < W.best_order))) {
        if (lane == 0) {
            W.best_score = score; W.best_order = order; W.best_n = cnt; W.best_buf = buf;
            atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
        }
    }
    __syncwarp();
}

// ---------------------------------------------------------------------------------------------
// Occurrence mode: ExpandSpeculationTree + SCORE for one (tree, p) job whose match node has at
// most 32 occurrences, a lane per occurrence.  cptr[k] (k >= 1) is the k-th token behind the
// lane's occurrence of the pattern and kmax says how many of them count (end of the text or
// sequence, depth cap; 0: the lane holds no occurrence of this job).
// A node below N_p is the set of lanes that agree on the tokens so far.  Every lane knows the
// deepest node on its own path that is already in the speculation tree (k levels down, index
// par_idx, D value d_par); the candidate it stands for is the next node on its path:
//   COUNT = lanes that agree on the next token too, sibling sum = lanes that have a next token.
// The candidates of all lanes together are exactly the frontier of Algorithm 1's expansion.
template <class BlockShared>
__device__ void expand_occ(BlockShared& sh, WarpWork& W, const int* cptr, int kmax, int tree, int p, int budget,
                           unsigned flags, int lane) {
    const int order = tree * SD_MAX_DEPTH + p;                  // loop order of Algorithm 1
    const int buf = W.best_buf ^ 1;
    int cnt = 0;
    double score = 0.0;
    bool dropped = false;
    int k = 0, par_idx = -1;
    double d_par = 1.0;                                         // D(N_p) = 1
    bool cv = false;                                            // this lane stands for a candidate
    int ctok = 0;
    double cd = 0.0;
    unsigned cmask = 0;                                         // lanes of the candidate node
    // candidates of the lanes in `grp`, which share (k, par_idx, d_par); returns the lanes with a next token
    auto refresh = [&](unsigned grp) -> unsigned {
        const bool in = (grp >> lane) & 1u;
        const bool valid = in && k + 1 <= kmax;
        const unsigned vm = __ballot_sync(FULL, valid);
        if (in) cv = false;
        if (valid) {
            ctok = cptr[k + 1];
            cmask = __match_any_sync(vm, ctok);
            const int c = __popc(cmask), s = __popc(vm);
            cd = c == s ? d_par : __dmul_rn(d_par, __ddiv_rn((double)c, (double)s));   // Eq. 2 with Eq. 1
            cv = true;
        }
        return vm;
    };
    refresh(__ballot_sync(FULL, kmax > 0));
    while (cnt < budget) {
        // ---- the best candidate: larger D, then smaller token, then smaller parent index
        const unsigned hi = cv ? (unsigned)__double2hiint(cd) : 0u;     // D > 0, so hi > 0 for a candidate
        const unsigned mx = __reduce_max_sync(FULL, hi);
        if (mx == 0u) break;                                    // the frontier is empty
        unsigned b = __ballot_sync(FULL, hi == mx);
        int leader = __ffs(b) - 1;
        unsigned lm = __shfl_sync(FULL, cmask, leader);
        if (b & ~lm) {                                          // several nodes share the high word: full comparison
            const bool in1 = hi == mx;
            const unsigned lo = in1 ? (unsigned)__double2loint(cd) : 0u;
            const unsigned mlo = __reduce_max_sync(FULL, lo);
            const bool in2 = in1 && lo == mlo;
            const unsigned mtk = __reduce_min_sync(FULL, in2 ? (unsigned)ctok : 0xffffffffu);
            const bool in3 = in2 && (unsigned)ctok == mtk;
            const unsigned mpk = __reduce_min_sync(FULL, in3 ? (unsigned)(par_idx + 1) : 0xffffffffu);
            b = __ballot_sync(FULL, in3 && (unsigned)(par_idx + 1) == mpk);
            leader = __ffs(b) - 1;
            lm = __shfl_sync(FULL, cmask, leader);
        }
        const double wd = __shfl_sync(FULL, cd, leader);
        const int wt = __shfl_sync(FULL, ctok, leader), wp = __shfl_sync(FULL, par_idx, leader);
        // everything still to come is at most wd each
        if ((score + (double)(budget - cnt) * wd) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
        if (lane == 0) { W.tok[buf][cnt] = wt; W.par[buf][cnt] = (unsigned char)(wp + 1); }
        score = __dadd_rn(score, wd);                           // Eq. 4, insertion order
        int idx = cnt++;
        const bool in = (lm >> lane) & 1u;
        if (in) { ++k; par_idx = idx; d_par = wd; }
        if ((flags & SD_FLAG_LINEAR) && !in) cv = false;        // chain variant: only the new node's children go on
        // the best of the other candidates: while the new node has one child that all its lanes
        // continue with, that child has the same D; if that is strictly above every other
        // candidate it is the next node whatever else there is, and no arg-max is needed
        const unsigned oth = __reduce_max_sync(FULL, (!in && cv) ? (unsigned)__double2hiint(cd) : 0u);
        const bool chain_ok = (unsigned)__double2hiint(wd) > oth;
        const int first = __ffs(lm) - 1;
        while (true) {
            const unsigned vm = refresh(lm);
            if (cnt >= budget || !chain_ok || vm != lm || __shfl_sync(FULL, cmask, first) != lm) break;
            if ((score + (double)(budget - cnt) * wd) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
            if ((lm & (lm - 1u)) == 0u) {
                // one occurrence: the rest of its text, as far as it counts and the budget goes
                const int k0 = __shfl_sync(FULL, k, first);
                const int len = min(__shfl_sync(FULL, kmax, first) - k0, budget - cnt);
                const int* src = (const int*)(unsigned long long)__shfl_sync(FULL, (unsigned long long)cptr, first);
                for (int j = lane; j < len; j += 32) {
                    W.tok[buf][cnt + j] = src[k0 + 1 + j];
                    W.par[buf][cnt + j] = (unsigned char)((j == 0 ? idx : cnt + j - 1) + 1);
                }
                for (int j = 0; j < len; ++j) score = __dadd_rn(score, wd);
                cnt += len;
                idx = cnt - 1;
                if (in) { k += len; par_idx = idx; }
            } else {
                const int ct = __shfl_sync(FULL, ctok, first);
                if (lane == 0) { W.tok[buf][cnt] = ct; W.par[buf][cnt] = (unsigned char)(idx + 1); }
                score = __dadd_rn(score, wd);
                idx = cnt++;
                if (in) { ++k; par_idx = idx; }
            }
        }
        if (dropped) break;
        // the final SCORE of this job is at least its running value: let the others prune on it
        if (lane == 0) atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
    }
    __syncwarp();
    if (!dropped && (score > W.best_score || (score == W.best_score && score > 0.0 && order < W.best_order))) {
        if (lane == 0) {
            W.best_score = score; W.best_order = order; W.best_n = cnt; W.best_buf = buf;
            atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
        }
    }
    __syncwarp();
}

// A per-request job that goes through the tree's entries: the match node of pattern length p is
// the slot's active node of depth p (kept current by the append).  Whole warp.
template <class BlockShared>
__device__ void request_tree_job(BlockShared& sh, WarpWork& W, const sd_store& sv, const SlotState* ss, const int4* s_ent, int t,
                                 int p, int budget, unsigned flags, int lane) {
    // an append that stopped early leaves a context the jobs were not made for
    if (ss->len != t || (ss->status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN))) return;
    int node = -1;
    unsigned rw = 0;
    if (lane == 0) {
        node = ss->active[p - 1];
        int rcb = ss->run_cb[p - 1];
        rw = ss->run_w[p - 1];
        if (node >= 0 && rw == RUN_UNKNOWN) { const int4 e = s_ent[node]; rcb = e.z; rw = (unsigned)e.w; }
        sh.node[1][p - 1] = node; sh.cb[1][p - 1] = rcb; sh.nc[1][p - 1] = rw;
    }
    node = __shfl_sync(FULL, node, 0);
    rw = (unsigned)__shfl_sync(FULL, rw, 0);
    __syncwarp();
    const int nch = (int)(rw & RUN_COUNT_MASK);
    if (node < 0 || nch == 0) return;
    if (nch > WIDE_RUN && !(rw & RUN_HAS_TOP)) {                 // scanned by all warps together, later
        if (lane == 0) sh.wide[atomicAdd(&sh.nwide, 1)] = SD_MAX_DEPTH + p - 1;
        return;
    }
    expand_job(sh, W, s_ent, (int)sv.spn, 1, p, budget, flags, false, 0, lane);
}

// One block of W warps per request.
//   1. match.  Global tree: the match nodes are advanced from the nodes cached at the previous
//      call by descending only the tokens appended since (full walks when the cache is stale).
//      Per-request tree: the slot's active nodes are the match nodes (sd_step: once the append
//      is done).  A block of sd_step that appends many tokens does not wait for that: it copies
//      the request's text (with the tokens being appended) into shared memory and scans it for the
//      earlier occurrences of its last token; the number of tokens before an occurrence that
//      agree with the context says which patterns it belongs to.
//   2. expand: the (tree, p) jobs that matched go into a queue, costliest first; a warp per job.
//      Global jobs go through the tree's entries.  Per-request jobs whose match node has at most
//      32 occurrences in a scanned text are read off the text (expand_occ: a lane per
//      occurrence, no tree) and come first; the others go through the request's tree from the
//      slot's active nodes.  sd_step: warp 0 appends the accepted tokens to the request's tree
//      meanwhile, exactly as sd_append would, and joins the queue when it is done; the other
//      warps meet at a barrier of their own until then, and only a warp that has taken a job
//      through the request's tree waits for the append (a bounded wait on a flag).
//   3. jobs of either tree that start at a wide child run without top block are scanned by all
//      warps together, behind a block-wide barrier.
//   4. select + emit from shared memory; no global scratch.
// A job is skipped or dropped, exactly, as soon as an upper bound of its SCORE falls below a
// score another job of the request has already reached (the running scores are published).
constexpr int BAR_GROUP = 1, BAR_JOIN = 2;    // hardware barriers beside the block-wide one

template <bool STEP, int WARPS, int MINB, int APPEND_G = 8>
__global__ void __launch_bounds__(WARPS * 32, MINB)
speculate_fused_kernel(sd_store sv, int n, const int32_t* __restrict__ d_slot, int Pe, double alpha, int max_spec,
                       unsigned flags, double tau, const int32_t* __restrict__ d_budget_cap, int32_t* d_n_draft,
                       int32_t* d_tokens, int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree,
                       int32_t* d_chosen_p, double* d_score, int32_t* d_status, const int64_t* __restrict__ d_app_off,
                       const int32_t* __restrict__ d_app_tok, int stage_tokens) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using BlockShared = BlockSharedT<WARPS>;
    constexpr int CTA_WARPS = WARPS;
    constexpr int NT = WARPS * 32;
    // the warps that do everything but the append: all of them, or all but warp 0
    constexpr int GW0 = STEP ? 1 : 0, GWARPS = WARPS - GW0, GT = GWARPS * 32;
    BlockShared& sh = *reinterpret_cast<BlockShared*>(smem_raw);
    int* const stx = reinterpret_cast<int*>(smem_raw + ((sizeof(BlockShared) + 15) & ~(size_t)15));
    // new tokens from which a block reads its text off shared memory: 6 with two blocks per SM
    // (9 warps scan), 12 with four (4 warps scan); measured, see the staging decision below
    constexpr int STAGE_MIN_NEW = MINB >= 4 ? 12 : 6;
    const int tid = threadIdx.x, lane = tid & 31, wib = tid >> 5;
    const int gtid = tid - GW0 * 32, gw = wib - GW0;             // index inside that group (negative: warp 0 of sd_step)
    auto group_sync = [&]() {
        if (STEP) asm volatile("bar.sync %0, %1;" ::"r"(BAR_GROUP), "r"(GT) : "memory");
        else __syncthreads();
    };
    const int i = blockIdx.x;
    const int M = sv.M, words = (M + 31) / 32, D = sv.D;
    const int slot = d_slot[i];
    const bool ok = slot >= 0 && slot < sv.R;
    // a slot may appear once per call: a later appearance is refused (two blocks on one tree would
    // race); the answer is collected at the first barrier below, before anything is written
    int dup = 0;
    for (int j = tid; j < i; j += NT) dup |= d_slot[j] == slot ? 1 : 0;
    int t = 0, status = SD_STATUS_BAD_SLOT;
    SlotState* ss = nullptr;
    if (ok) { ss = sv.s_state + slot; t = ss->len; status = ss->status; }
    // STEP: t_old tokens are in the slot's text, the next n_new come from the append list; the
    // match below already runs on the context of t = t_old + n_new tokens
    const int t_old = t;
    const int32_t* newtok = nullptr;
    int n_new = 0;
    if (STEP && ok) {
        newtok = d_app_tok + d_app_off[i];
        n_new = (int)(d_app_off[i + 1] - d_app_off[i]);
        t = t_old + n_new;
    }
    bool usable = ok && !(status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN)) && t > 0;
    // the stored text starts its way into shared memory now (asynchronous copies, nothing waits
    // for them here): it arrives while the cached match nodes and the append list are read
    const int32_t* text = ok ? sv.s_text + (long long)slot * sv.T : nullptr;
    const bool prefetched = STEP && MINB > 1 && n_new >= STAGE_MIN_NEW && ok && gtid >= 0 && t_old <= stage_tokens && !(flags & SD_FLAG_GLOBAL_ONLY);
    if (prefetched) {
        const unsigned dst0 = (unsigned)__cvta_generic_to_shared(stx);
        for (int q = gtid; q < t_old; q += GT)
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst0 + 4u * q), "l"(text + q) : "memory");
    }
    int cap = max_spec;
    if (d_budget_cap && d_budget_cap[i] >= 0) cap = min(cap, d_budget_cap[i]);
    if (tid < 2 * SD_MAX_DEPTH) { (&sh.node[0][0])[tid] = -1; (&sh.nc[0][0])[tid] = 0; }
    if (tid < SD_MAX_DEPTH + 2) { sh.r_hist[tid] = 0; sh.r_cum[tid] = 0; sh.r_fill[tid] = 0; }
    if (tid == 0) {
        sh.njobs = 0; sh.next = 0; sh.nwide = 0; sh.nwide_kept = 0; sh.best_hi = 0u; sh.win_warp = -1;
        sh.r_pn = SD_MAX_DEPTH + 1; sh.scan_next[0] = 0; sh.scan_next[1] = 0; sh.app_done = 0; sh.nlate = 0;
    }
    WarpWork& W = sh.w[wib];
    if (lane == 0) { W.best_score = 0.0; W.best_order = 1 << 30; W.best_n = 0; W.best_buf = 0; }

    // ---------------- 1. match
    bool want_g = usable && !(flags & SD_FLAG_REQUEST_ONLY);
    bool want_r = usable && !(flags & SD_FLAG_GLOBAL_ONLY);
    // warps that advance the global match nodes, and this warp's rank among them
    const int mwarps = GWARPS;
    const int mrank = gw;
    constexpr int MROUNDS = (SD_MAX_DEPTH + GWARPS - 1) / GWARPS;   // pattern lengths per warp
    int src_node[MROUNDS], src_from[MROUNDS];                   // per target: start node and first text index
#pragma unroll
    for (int h = 0; h < MROUNDS; ++h) { src_node[h] = -1; src_from[h] = 0; }
    if (want_g && mrank >= 0) {
        const bool cache_ok = ss->g_gen == ss->gen && ss->g_epoch == sv.g_state->epoch && ss->g_len <= t;
        const int k = t - ss->g_len;                            // tokens appended since the cache was taken
        const int depths = ss->g_depths;
#pragma unroll
        for (int h = 0; h < MROUNDS; ++h) {
            const int d = mrank + 1 + h * mwarps;               // target pattern length
            if (d > Pe || d > t) continue;
            if (cache_ok && d > k && d - k <= depths) {
                src_node[h] = ss->g_node[d - k - 1];            // node of the tokens before the new ones
                src_from[h] = t - k;
            } else {
                const int x0 = t - d < t_old ? text[t - d] : newtok[t - d - t_old];
                src_node[h] = (x0 >= 0 && x0 < sv.V) ? sv.g_root[x0] : -1;
                src_from[h] = t - d + 1;
            }
        }
    }
    // all cached nodes read before any is replaced; and: is this a second block for the same slot?
    const bool refused = __syncthreads_or(dup) != 0;
    if (refused) { usable = false; want_g = false; want_r = false; status = SD_STATUS_BAD_SLOT; }
    // The text can be read off only if it fits the shared memory left for it, and it is only
    // worth the copy and the scan (about 16 us for 4,096 tokens) where a long append would
    // otherwise hold the per-request jobs up: from STAGE_MIN_NEW new tokens on.  sd_speculate
    // does not read it at all: with no append going on, the slot's active nodes are the
    // per-request match nodes, at no cost.  Nor do blocks that have an SM to themselves (small
    // batches: measured on 64 requests with 8,192-token texts, 112 us per step without, 141 with).
    const bool staged = STEP && MINB > 1 && n_new >= STAGE_MIN_NEW && want_r && t >= 2 && t <= stage_tokens;
    const int Lcap = min(Pe, D - 1);                            // a match node at depth D has no children
    if (STEP && wib == 0) {
        if (ok && n_new > 0 && !refused) {
            // ---- the request's accepted tokens go into its tree and text (as sd_append does)
            int32_t* wtext = sv.s_text + (long long)slot * sv.T;
            TreeRef tr{sv.s_ent + (long long)slot * sv.spn, sv.s_root + (long long)slot * sv.V, (int)sv.spn};
            int len = ss->len, used = ss->used, live = ss->live, st = ss->status;
            int act = ss->active[lane], room = ss->room[lane], run_cb = ss->run_cb[lane];
            unsigned run_w = ss->run_w[lane];
            for (int k = 0; k < n_new && !(st & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN)); ++k) {
                const int x = newtok[k];
                if (x < 0 || x >= sv.V) { st |= SD_STATUS_BAD_TOKEN; break; }
                if (len >= sv.T || !append_token<APPEND_G>(tr, sv.D, x, len, lane, act, room, run_cb, run_w, used, live)) {
                    st |= SD_STATUS_POOL_FULL;
                    break;
                }
                if (lane == 0) wtext[len] = x;
                ++len;
            }
            ss->active[lane] = act; ss->room[lane] = room; ss->run_cb[lane] = run_cb; ss->run_w[lane] = run_w;
            if (lane == 0) { ss->len = len; ss->used = used; ss->live = live; ss->status = st; }
        }
        __threadfence_block();
        if (lane == 0) *(volatile int*)&sh.app_done = 1;        // the jobs that go through the tree may start
        // join the others once their queue is ready
        asm volatile("bar.sync %0, %1;" ::"r"(BAR_JOIN), "r"(NT) : "memory");
    } else {
        // ---- the tokens being appended join the text in shared memory
        if (staged)
            for (int q = t_old + gtid; q < t; q += GT) stx[q] = newtok[q - t_old];
        // ---- global match nodes
        if (want_g) {
#pragma unroll
            for (int h = 0; h < MROUNDS; ++h) {
                const int d = mrank + 1 + h * mwarps;
                if (d > Pe) continue;
                int cb = 0;
                unsigned wf = 0;
                const int node = (d > t) ? -1 : walk_from(sv.g_ent, (int)sv.g_cap, src_node[h], text, t_old, newtok, src_from[h], t,
                                                          lane, cb, wf);
                if (lane == 0) {
                    ss->g_node[d - 1] = node;
                    sh.node[0][d - 1] = node;
                    if (node >= 0) { sh.cb[0][d - 1] = cb; sh.nc[0][d - 1] = wf; }
                }
            }
            if (gtid == 0) { ss->g_gen = ss->gen; ss->g_epoch = sv.g_state->epoch; ss->g_len = t; ss->g_depths = Pe; }
        }
        if (prefetched) asm volatile("cp.async.wait_all;" ::: "memory");
        group_sync();                                           // the text is in shared memory
        // ---- per-request occurrences: a chunk of 256 positions at a time, handed out by a counter
        // (warps that come late from their walks take fewer).  Pass 0 finds the occurrences of the
        // last token, notes their match lengths and counts them by length; pass 1 collects those
        // of the patterns that have at most 32 of them.
        const int last = staged ? stx[t - 1] : 0;
        const int nchunks = staged ? (t - 1 + 255) / 256 : 0;
        unsigned char* const sell = reinterpret_cast<unsigned char*>(stx + stage_tokens);   // match length per position (0: none)
        auto scan_pass = [&](int pass) {
            const int pn = sh.r_pn;
            while (true) {
                int c = 0;
                if (lane == 0) c = atomicAdd(&sh.scan_next[pass], 1);
                c = __shfl_sync(FULL, c, 0);
                if (c >= nchunks) break;
#pragma unroll 1
                for (int u = 0; u < 8; ++u) {
                    const int e = c * 256 + u * 32 + lane;
                    if (e >= t - 1) continue;
                    if (pass == 0) {
                        int l = 0;
                        if (stx[e] == last) {
                            l = 1;
                            while (l < Lcap && e - l >= 0 && stx[e - l] == stx[t - 1 - l]) ++l;
                            // equal lengths of the 32 positions are counted once (frequent last tokens
                            // would otherwise all queue up at one counter)
                            const unsigned grp = __match_any_sync(__activemask(), l);
                            if (lane == __ffs(grp) - 1) atomicAdd(&sh.r_hist[l], __popc(grp));
                        }
                        sell[e] = (unsigned char)l;
                    } else {
                        const int l = sell[e];
                        if (l >= pn) sh.r_list[sh.r_cum[l + 1] + atomicAdd(&sh.r_fill[l], 1)] = e;
                    }
                }
            }
        };
        scan_pass(0);
        group_sync();
        if (gw == 0) {
            int h = (lane + 1 <= Lcap) ? sh.r_hist[lane + 1] : 0;   // lane L: matches of exactly L + 1 tokens
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {                  // suffix sums: matches of at least L + 1 tokens
                const int y = __shfl_down_sync(FULL, h, o);
                if (lane + o < 32) h += y;
            }
            sh.r_cum[lane + 1] = h;
            const unsigned few = __ballot_sync(FULL, h <= SD_OCC_LANES);
            if (lane == 0) sh.r_pn = __ffs(few);                // (the counts fall with the length: lane 31 always qualifies)
        }
        group_sync();
        if (staged && sh.r_cum[sh.r_pn] > 0) scan_pass(1);
        group_sync();

        // ---------------- 2. the job queue, costliest first.  Per-request jobs that have to go through
        // the tree (more than 32 occurrences, or no text in shared memory) come last: in sd_step
        // they have to wait for the append.
        // (order: the jobs that are read off the text first: they are quick and a long match there
        // sets a score that rules out most of the others; then by the nodes a job can add at most)
        if (gtid < 2 * SD_MAX_DEPTH) {
            const int tree = gtid / SD_MAX_DEPTH, p = gtid % SD_MAX_DEPTH + 1;
            int c = 0;
            if (tree == 0) {
                const unsigned wf = sh.nc[0][p - 1];
                const int nch = (int)(wf & RUN_COUNT_MASK);
                if (p <= Pe && sh.node[0][p - 1] >= 0 && nch > 0) {
                    // all first runs start their way to L2 now, long before a warp gets to them
                    const int4* base = sv.g_ent + sh.cb[0][p - 1];
                    const int lines = min(4, (nch + 7) >> 3);
                    for (int l = 0; l < lines; ++l) prefetch_l2(base + l * 8);
                    c = min(budget_for(alpha, p, cap), 2 * (D - p));
                    if (c > 0 && nch > WIDE_RUN && !(wf & RUN_HAS_TOP)) { sh.wide[atomicAdd(&sh.nwide, 1)] = gtid; c = 0; }
                    if (c > 0) c += 1000;
                }
            } else if (want_r && p <= Pe && p <= t) {
                c = min(budget_for(alpha, p, cap), 2 * (D - p));
                if (staged && !(p <= Lcap && sh.r_cum[p] > 0)) c = 0;      // no earlier occurrence: nothing to speculate
                else if (c > 0 && staged && p >= sh.r_pn) c += 2000;       // read off the text
                else if (c > 0) c += 1000;                                  // through the request's tree: by cost among the global jobs
            }
            sh.cost[gtid] = c;
        }
        group_sync();
        if (gtid < 2 * SD_MAX_DEPTH) {
            const int c = sh.cost[gtid];
            if (c > 0) {
                int rank = 0;
                for (int q = 0; q < 2 * SD_MAX_DEPTH; ++q) {
                    const int cq = sh.cost[q];
                    rank += (cq > c || (cq == c && q < gtid)) ? 1 : 0;
                }
                sh.job[rank] = gtid | ((c < 2000 && gtid >= SD_MAX_DEPTH) ? 128 : 0);   // bit 7: through the request's tree (sd_step: once the append is done)
                atomicAdd(&sh.njobs, 1);
            }
        }
        group_sync();
        if (STEP) asm volatile("bar.arrive %0, %1;" ::"r"(BAR_JOIN), "r"(NT) : "memory");   // warp 0 may come in
    }
    const int4* s_ent = ok ? sv.s_ent + (long long)slot * sv.spn : nullptr;
    {
        const int njobs = sh.njobs;
        while (true) {
            int j = 0;
            if (lane == 0) j = atomicAdd(&sh.next, 1);
            j = __shfl_sync(FULL, j, 0);
            if (j >= njobs) break;
            const int code = sh.job[j];
            const int tree = (code & 127) / SD_MAX_DEPTH, p = (code & 127) % SD_MAX_DEPTH + 1;
            const int budget = budget_for(alpha, p, cap);
            // SCORE <= number of draft nodes (every D <= 1), and SCORE <= number of levels below the
            // match node: the D values of one level of a tree add up to at most 1 (Eq. 1 shares out
            // the parent's D among its children)
            if ((double)min(budget, D - p) * 1.000000001 < best_so_far(sh)) continue;
            if (tree == 0) {
                expand_job(sh, W, sv.g_ent, (int)sv.g_cap, 0, p, budget, flags, false, 0, lane);
            } else if (!(code & 128)) {
                const int m = sh.r_cum[p];
                const int e = lane < m ? sh.r_list[lane] : 0;
                const int kmax = lane < m ? min(t - 1 - e, D - p) : 0;
                expand_occ(sh, W, stx + e, kmax, 1, p, budget, flags, lane);
            } else {
                // through the tree: the match node is the slot's active node of depth p, once the
                // append is done (bounded wait; a job that runs out of patience is done after the
                // block-wide barrier below instead)
                bool ready = true;
                if (STEP) {
                    ready = false;
                    for (int spin = 0; spin < 4096 && !ready; ++spin) {
                        int flag = 0;
                        if (lane == 0) flag = *(volatile int*)&sh.app_done;
                        ready = __shfl_sync(FULL, flag, 0) != 0;
                        if (!ready) __nanosleep(200);
                    }
                }
                if (!ready) { if (lane == 0) sh.late[atomicAdd(&sh.nlate, 1)] = p; continue; }
                request_tree_job(sh, W, sv, ss, s_ent, t, p, budget, flags, lane);
            }
        }
    }
    __syncthreads();                                            // sd_step: the append is done and visible

    // ---------------- 3. what had to wait: an append that stopped early, per-request jobs whose wait
    // ran out, jobs that start at a wide child run
    if (STEP && ok && !refused) {
        status = ss->status;
        if (ss->len != t || (status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN))) {
            // the append stopped early: no speculation for this request, and the match nodes
            // taken above describe a context that does not exist
            usable = false; want_g = false; want_r = false;
            t = ss->len;
            if (tid == 0) ss->g_gen = ss->gen - 1;
        }
    }
    for (int q = wib; q < sh.nlate && usable; q += CTA_WARPS) {
        const int p = sh.late[q];
        const int budget = budget_for(alpha, p, cap);
        if ((double)min(budget, D - p) * 1.000000001 < best_so_far(sh)) continue;
        request_tree_job(sh, W, sv, ss, s_ent, t, p, budget, flags, lane);
    }
    __syncthreads();
    // Jobs that start at a wide node (short patterns, hence small budgets): most cannot reach
    // the best score any more and are dropped here.  For the rest the warps of the block share
    // the scan of the run, then one warp merges the partial lists and finishes the job.
    if (tid == 0) {
        const double best = __hiloint2double((int)sh.best_hi, 0);
        int kept = 0;
        for (int q = 0; q < sh.nwide && usable; ++q) {
            const int p = sh.wide[q] % SD_MAX_DEPTH + 1;
            if (!((double)min(budget_for(alpha, p, cap), D - p) * 1.000000001 < best)) sh.wide[kept++] = sh.wide[q];
        }
        sh.nwide_kept = kept;
    }
    __syncthreads();
    const int nwide = sh.nwide_kept;
    for (int base = 0; base < nwide; base += CTA_WARPS) {
        const int nj = min(CTA_WARPS, nwide - base);
        const int G = CTA_WARPS / nj;                           // warps per job
        const int my_job = wib / G, my_slice = wib % G;
        const bool active = my_job < nj;
        int tree = 0, p = 1, budget = 0, fs = 0;
        const int4* ent = sv.g_ent;
        if (active) {
            const int code = sh.wide[base + my_job];
            tree = code / SD_MAX_DEPTH; p = code % SD_MAX_DEPTH + 1;
            budget = budget_for(alpha, p, cap);
            ent = tree == 0 ? sv.g_ent : s_ent;
            long long sum;
            scan_run_by_count(ent, sh.cb[tree][p - 1], (int)(sh.nc[tree][p - 1] & RUN_COUNT_MASK), my_slice, G, -1, 1, W,
                              W.F, 0, fs, budget, sum, lane);
            if (lane == 0) { sh.slice_sum[wib] = sum; sh.slice_fs[wib] = fs; }
        }
        __syncthreads();
        if (active && my_slice == 0) {
            long long sum = sh.slice_sum[wib];
            for (int g = 1; g < G; ++g) {
                const Frontier& O = sh.w[wib + g].F;
                const int ofs = sh.slice_fs[wib + g];
                sum += sh.slice_sum[wib + g];
                frontier_merge_list(W.F, 0, fs, budget, O, ofs, -1, lane);
            }
            counts_to_d(W.F, 0, fs, 1.0, sum, lane);
            expand_job(sh, W, ent, tree == 0 ? (int)sv.g_cap : (int)sv.spn, tree, p, budget, flags, true, fs, lane);
        }
        __syncthreads();
    }

    // ---------------- 4. select (first in loop order among the largest scores) and emit
    if (wib == 0) {
        double sc = lane < CTA_WARPS ? sh.w[lane].best_score : 0.0;
        int od = lane < CTA_WARPS ? sh.w[lane].best_order : 1 << 30;
        int ww = lane;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const double osc = __shfl_xor_sync(FULL, sc, off);
            const int ood = __shfl_xor_sync(FULL, od, off);
            const int oww = __shfl_xor_sync(FULL, ww, off);
            if (osc > sc || (osc == sc && ood < od)) { sc = osc; od = ood; ww = oww; }
        }
        // Section 3.2: the tree is used only if its score exceeds the threshold (tau = 0: any score above 0)
        if (lane == 0) sh.win_warp = (usable && sc > 0.0 && sc > tau) ? ww : -1;
    }
    __syncthreads();
    const int win = sh.win_warp;
    int nd = 0, ctree = -1, cp = 0;
    double best = 0.0;
    const int* wtok = nullptr;
    const unsigned char* wpar = nullptr;
    if (win >= 0) {
        const WarpWork& B = sh.w[win];
        nd = B.best_n; best = B.best_score;
        ctree = B.best_order / SD_MAX_DEPTH; cp = B.best_order % SD_MAX_DEPTH;
        if (cp == 0) { cp = SD_MAX_DEPTH; ctree -= 1; }          // order = tree * 32 + p with p in 1..32
        wtok = B.tok[B.best_buf]; wpar = B.par[B.best_buf];
    }
    for (int j = tid; j < M; j += NT) {
        int tok = -1, par = -1, pos = -1;
        unsigned long long bits = 0;
        if (j < nd) {
            tok = wtok[j];
            par = (int)wpar[j] - 1;
            int depth = 0;
            for (int a = j, hops = 0; a >= 0 && hops < SD_MAX_SPEC; a = (int)wpar[a] - 1, ++hops) {
                bits |= 1ull << a;
                ++depth;
            }
            pos = t + depth - 1;
        }
        const long long o = (long long)i * M + j;
        d_tokens[o] = tok; d_parents[o] = par; d_positions[o] = pos;
        d_mask[o * words] = (uint32_t)bits;
        if (words > 1) d_mask[o * words + 1] = (uint32_t)(bits >> 32);
    }
    if (tid == 0) {
        d_n_draft[i] = nd; d_chosen_tree[i] = ctree; d_chosen_p[i] = cp; d_score[i] = best;
        if (d_status) d_status[i] = status;
    }
}

}  // namespace

namespace {

constexpr int SMEM_PER_SM = 228 * 1024;       // shared memory of one SM; a resident block also costs 1 KB of it
constexpr int MAX_DEVICES = 64;
struct DeviceInfo { bool ready = false; int sm_count = 0; };
DeviceInfo g_dev[MAX_DEVICES];
std::mutex g_dev_mutex;

// tokens of text a block of this shape can hold in shared memory beside its working set
template <int WARPS, int MINB>
constexpr int stage_limit_tokens() {
    return (int)((SMEM_PER_SM / MINB - 1024 - (int)((sizeof(BlockSharedT<WARPS>) + 15) & ~(size_t)15)) / 5) & ~15;   // 4 + 1 bytes per token
}

template <bool STEP, int WARPS, int MINB, int G>
int raise_smem_limit() {
    return cudaFuncSetAttribute(speculate_fused_kernel<STEP, WARPS, MINB, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                SMEM_PER_SM / MINB - 1024) == cudaSuccess ? SD_OK : SD_ERR_CUDA;
}

// once per device: raise the kernels' dynamic shared memory limit, read the SM count
int device_setup(int dev, int* sm_count) {
    if (dev < 0 || dev >= MAX_DEVICES) return SD_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_dev[dev].ready) {
        if (raise_smem_limit<false, CTA_WARPS, 2, 8>() != SD_OK || raise_smem_limit<true, CTA_WARPS_STEP, 2, STEP_G>() != SD_OK ||
            raise_smem_limit<false, CTA_WARPS_WIDE, 1, 8>() != SD_OK || raise_smem_limit<true, CTA_WARPS_WIDE_STEP, 1, 8>() != SD_OK ||
            raise_smem_limit<false, CTA_WARPS_NARROW, 4, 8>() != SD_OK ||
            raise_smem_limit<true, CTA_WARPS_NARROW_STEP, 4, STEP_G>() != SD_OK)
            return SD_ERR_CUDA;
        SD_CUDA_OK(cudaDeviceGetAttribute(&g_dev[dev].sm_count, cudaDevAttrMultiProcessorCount, dev));
        g_dev[dev].ready = true;
    }
    *sm_count = g_dev[dev].sm_count;
    return SD_OK;
}

}  // namespace

static int launch_fused(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm,
                        const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents,
                        int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
                        double* d_score, int32_t* d_status, const int64_t* d_app_off, const int32_t* d_app_tok,
                        bool step, void* stream) {
    if (!s || !prm || n < 0 || n > s->R) return SD_ERR_INVALID_ARG;
    if (prm->P < 1 || prm->max_spec < 0 || prm->max_spec > s->M || !(prm->alpha >= 0.0) || !(prm->tau >= 0.0))
        return SD_ERR_INVALID_ARG;
    if ((prm->flags & SD_FLAG_GLOBAL_ONLY) && (prm->flags & SD_FLAG_REQUEST_ONLY)) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    if (n == 0) return SD_OK;
    if (!d_slot || !d_n_draft || !d_tokens || !d_parents || !d_positions || !d_mask || !d_chosen_tree || !d_chosen_p ||
        !d_score)
        return SD_ERR_INVALID_ARG;
    if (step && !d_app_off) return SD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int Pe = prm->P < s->D ? prm->P : s->D;               // longer patterns never match
    int sms = 0;
    const int rc = device_setup(s->device, &sms);
    if (rc != SD_OK) return rc;
    // one block per SM is all a small batch can use: sd_speculate then takes more warps if a
    // request has more jobs (two trees, Pe pattern lengths each) than 16 warps start at once,
    // sd_step takes more registers
    const bool wide = n <= sms && (step || 2 * Pe > 2 * CTA_WARPS);
    // more requests than two 16-warp blocks per SM hold at once: smaller blocks, one wave
    const bool narrow = n > 2 * sms;
    // Behind its working set a block keeps the request's text in shared memory if it fits (a
    // longer text is not scanned: all of its per-request jobs go through the tree).
#define SD_LAUNCH_FUSED(STEP, WARPS, MINB, G, OFF, TOK)                                                                 \
    do {                                                                                                                 \
        const int lim = stage_limit_tokens<WARPS, MINB>();                                                               \
        const int stage = s->T <= lim ? ((s->T + 15) & ~15) : 0;                                                         \
        const size_t smem = ((sizeof(BlockSharedT<WARPS>) + 15) & ~(size_t)15) + (size_t)stage * 5;                      \
        speculate_fused_kernel<STEP, WARPS, MINB, G><<<(unsigned)n, WARPS * 32, smem, st>>>(                             \
            *s, n, d_slot, Pe, prm->alpha, prm->max_spec, prm->flags, prm->tau, d_budget_cap, d_n_draft, d_tokens,       \
            d_parents, d_positions, d_mask, d_chosen_tree, d_chosen_p, d_score, d_status, OFF, TOK, stage);              \
    } while (0)
    if (step) {
        if (wide) SD_LAUNCH_FUSED(true, CTA_WARPS_WIDE_STEP, 1, 8, d_app_off, d_app_tok);
        else if (narrow) SD_LAUNCH_FUSED(true, CTA_WARPS_NARROW_STEP, 4, STEP_G, d_app_off, d_app_tok);
        else SD_LAUNCH_FUSED(true, CTA_WARPS_STEP, 2, STEP_G, d_app_off, d_app_tok);
    } else {
        if (wide) SD_LAUNCH_FUSED(false, CTA_WARPS_WIDE, 1, 8, nullptr, nullptr);
        else if (narrow) SD_LAUNCH_FUSED(false, CTA_WARPS_NARROW, 4, 8, nullptr, nullptr);
        else SD_LAUNCH_FUSED(false, CTA_WARPS, 2, 8, nullptr, nullptr);
    }
#undef SD_LAUNCH_FUSED
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}

extern "C" int sd_speculate(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm,
                            const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents,
                            int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
                            double* d_score, int32_t* d_status, void* stream) {
    return launch_fused(s, n, d_slot, prm, d_budget_cap, d_n_draft, d_tokens, d_parents, d_positions, d_mask, d_chosen_tree,
                        d_chosen_p, d_score, d_status, nullptr, nullptr, false, stream);
}

extern "C" int sd_step(sd_store* s, int32_t n, const int32_t* d_slot, const int64_t* d_offsets, const int32_t* d_new_tokens,
                       const sd_spec_params* prm, const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens,
                       int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree,
                       int32_t* d_chosen_p, double* d_score, int32_t* d_status, void* stream) {
    return launch_fused(s, n, d_slot, prm, d_budget_cap, d_n_draft, d_tokens, d_parents, d_positions, d_mask, d_chosen_tree,
                        d_chosen_p, d_score, d_status, d_offsets, d_new_tokens, true, stream);
}

// ---------------------------------------------------------------------------------------------
// sd_speculate_noalloc: the same two kernels, with the per-job scratch records kept in a
// fixed array that is part of the loaded library image instead of in memory obtained
// from cudaMalloc.  Meant for callers that must not touch the CUDA allocator at all
// (see the declaration in suffixspec.h).
//
// The array's name below is only meaningful to device code.  Host code holds a stand-in
// symbol of the same name, so the launch code first asks the runtime for the array's
// real device address (once per device, with that device current) and passes that on.
namespace {

constexpr long long NOALLOC_BYTES =
    (long long)SD_NOALLOC_MAX_JOBS * (sizeof(double) + sizeof(int32_t) + 2ll * SD_MAX_SPEC * sizeof(int32_t));

static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
unsigned char* g_noalloc_ptr[NOALLOC_MAX_DEVICES];      // device address of the array, per device
bool g_noalloc_ready[NOALLOC_MAX_DEVICES];
std::mutex g_noalloc_mutex;

// Device address of the scratch array on the current device (looked up on first use).
int noalloc_scratch_address(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return SD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ready[dev]) {
        unsigned char* p = nullptr;
        if (cudaGetSymbolAddress((void**)&p, g_noalloc_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return SD_ERR_CUDA;
        }
        g_noalloc_ptr[dev] = p;
        g_noalloc_ready[dev] = true;
    }
    *out = g_noalloc_ptr[dev];
    return SD_OK;
}

}  // namespace

extern "C" int sd_speculate_noalloc(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm,
                                    const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens,
                                    int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree,
                                    int32_t* d_chosen_p, double* d_score, int32_t* d_status, void* stream) {
    if (!s || !prm || n < 0 || n > s->R) return SD_ERR_INVALID_ARG;
    if (prm->P < 1 || prm->max_spec < 0 || prm->max_spec > s->M || !(prm->alpha >= 0.0) || !(prm->tau >= 0.0))
        return SD_ERR_INVALID_ARG;
    if ((prm->flags & SD_FLAG_GLOBAL_ONLY) && (prm->flags & SD_FLAG_REQUEST_ONLY)) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    // one record per (request, tree, depth): the batch must fit the fixed array
    if ((long long)n * 2 * s->D > SD_NOALLOC_MAX_JOBS) return SD_ERR_CAPACITY;
    if (n == 0) return SD_OK;
    if (!d_slot || !d_n_draft || !d_tokens || !d_parents || !d_positions || !d_mask || !d_chosen_tree || !d_chosen_p ||
        !d_score)
        return SD_ERR_INVALID_ARG;
    unsigned char* base = nullptr;
    const int rc = noalloc_scratch_address(&base);
    if (rc != SD_OK) return rc;
    // Same record layout as the store's own scratch, carved out of the fixed array.  Every
    // record the second kernel reads is written by the first kernel of the same call, so
    // nothing left over from an earlier call is ever consumed and nothing needs clearing.
    sd_store view = *s;
    view.j_score = reinterpret_cast<double*>(base);
    view.j_n = reinterpret_cast<int32_t*>(base + (long long)SD_NOALLOC_MAX_JOBS * sizeof(double));
    view.j_tok = view.j_n + SD_NOALLOC_MAX_JOBS;
    view.j_par = view.j_tok + (long long)SD_NOALLOC_MAX_JOBS * SD_MAX_SPEC;
    cudaStream_t st = (cudaStream_t)stream;
    const int Pe = prm->P < s->D ? prm->P : s->D;
    const long long jobs = (long long)n * 2 * Pe;
    match_expand_kernel<<<(unsigned)((jobs + SPEC_WARPS - 1) / SPEC_WARPS), SPEC_WARPS * 32, 0, st>>>(
        view, n, d_slot, Pe, prm->alpha, prm->max_spec, prm->flags, d_budget_cap);
    select_emit_kernel<<<(unsigned)((n + 3) / 4), 128, 0, st>>>(view, n, d_slot, Pe, prm->tau, d_n_draft, d_tokens, d_parents,
                                                                d_positions, d_mask, d_chosen_tree, d_chosen_p, d_score,
                                                                d_status);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
