// GenerateCandidateTree (Algorithm 1) for a whole batch: one thread block per request, one
// launch per decode step (sd_step: the accepted tokens are appended in the same launch).
//
//   1. text.  The request's text x_{1:t} is copied into shared memory (new tokens included).
//   2. match.
//      Per-request tree (implicit, see common.cuh): the block scans the text for the earlier
//      occurrences of the last token and measures, for each, how many tokens before it agree
//      with the context (at most P).  Sorted by that length, the occurrences of the pattern of
//      length p are a prefix of the list: that prefix IS the match node N_p.
//      Global tree: MatchPattern walks from the root table, the shortest patterns first, a warp
//      per pattern length, until a match node has at most 32 occurrences and was never touched
//      by an online insert.  Such a node is a range of the offline build's suffix order; its
//      occurrences are read from there with the text around them (64 tokens each), and the
//      occurrences of every longer pattern are those among them whose preceding tokens agree
//      with the context.  No longer pattern is walked.
//   3. expand.  The (tree, p) jobs that matched go into a queue, costliest first; a warp per job.
//      Occurrence mode (at most 32 occurrences): a lane per occurrence.  A node of the suffix
//      tree below N_p is the set of lanes whose next tokens agree so far, its count their number
//      (Eq. 1 and Eq. 2 from popcounts), and the frontier of ExpandSpeculationTree is "the next
//      node on every lane's path": the best candidate is a warp-wide arg-max, adding it moves
//      its lanes one token on.  Chains are added without an arg-max.
//      Wide per-request nodes (more than 32 occurrences: short patterns of frequent tokens, small
//      budgets): children by a histogram of the next tokens over the occurrence list.
//      Global nodes with more than 32 occurrences or touched by an insert: the tree's entries
//      (sorted child runs, top blocks, windows of 32 entries) with a sorted frontier.
//      A job is dropped, exactly, as soon as an upper bound of its SCORE (every D <= 1 and D
//      never grows along a path) falls below a score another job of the request has reached.
//   4. select (first in loop order among the largest scores; Section 3.2: only if SCORE > tau)
//      and emit tokens, parents, positions and the tree-attention mask.
//
// fp64 rules: C = count / sibling-sum (Eq. 1), D = D(parent) * C (Eq. 2), SCORE
// adds D in insertion order; __ddiv_rn / __dmul_rn / __dadd_rn keep every
// operation a separately rounded IEEE binary64 operation (no FMA contraction).
#include <mutex>

#include "common.cuh"
#include "suffix_order.cuh"

namespace {

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

__device__ __forceinline__ int budget_for(double alpha, int p, int cap) {
    const double b = floor(__dmul_rn(alpha, (double)p));        // Eq. 3
    if (b > (double)cap) return cap;
    if (b < 0.0) return 0;
    return (int)b;
}

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
    int node[2][SD_MAX_DEPTH];                // global tree: match node per pattern length (-1: none); row 1 unused
    int cb[2][SD_MAX_DEPTH];                  // its child run
    unsigned nc[2][SD_MAX_DEPTH];             // ... as the node's w field (count | flags)
    int cost[2 * SD_MAX_DEPTH];
    int job[2 * SD_MAX_DEPTH];
    int wide[2 * SD_MAX_DEPTH];               // jobs whose match node has a wide child run
    int njobs, next, nwide, nwide_kept;
    long long slice_sum[WARPS];
    int slice_fs[WARPS];
    unsigned best_hi;                         // high word of the largest SCORE reached so far: a lower
                                              // bound of it (scores are non-negative doubles), which is
                                              // all the pruning needs; 32 bits keep the atomic native
    int win_warp;
    int first_bad;                            // sd_step: first new token outside the vocabulary
    // per-request tree: the match nodes as ranges of the text's suffix order
    int r_lo[SD_MAX_DEPTH + 1];               // r_lo[p]: first suffix that starts with the last p tokens (the context's own end)
    int r_cnt[SD_MAX_DEPTH + 1];              // earlier occurrences of that pattern: suffixes r_lo[p] + 1 .. r_lo[p] + r_cnt[p]
    SaTemp sat;                               // scratch of the suffix-order update
    // global tree: the base of occurrence mode
    int g_cnt[SD_MAX_DEPTH];                  // COUNT of the match node
    int g_rank[SD_MAX_DEPTH];                 // its first suffix in the suffix order (-1: not usable as base)
    int g_walked, g_failed, g_base_p, g_base_m;
    int g_src[SD_MAX_DEPTH];                  // the slot's cached match nodes, as they were before this launch
    int g_src_depths, g_src_k;                // how many are cached (0: none usable), tokens appended since
    int g_pos[SD_OCC_BASE];                   // text position of the occurrence's first pattern token
    int g_ell[SD_OCC_BASE];                   // longest pattern the occurrence matches
    int g_avail[SD_OCC_BASE];                 // tokens that follow the pattern inside the sequence (depth cap applied)
    int g_cum[SD_MAX_DEPTH + 2];
    int gwin[SD_OCC_BASE][64];                // tokens pos - 32 .. pos + 31 around every occurrence
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
    // D = d_parent * count / sum, so small counts lose without any fp64 work.
    double need = 0.0;
    if (fs == K) {
        const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
        need = F.d[last] * dsum * 0.999999;                     // count * d_parent must reach this
    }
    for (int base = 0; base < n; base += 32) {
        const int idx = base + lane;
        int4 e = w;
        if (base != 0) { e = make_int4(0, 0, 0, 0); if (idx < n) e = ent[cb + idx]; }
        bool pass = idx < n && idx != skip && (double)e.y * d_parent >= need;
        if (!__any_sync(FULL, pass)) continue;
        if (fs == 0 && n <= 32) {
            // Nothing waits yet (the first children of a job): the candidates are siblings, and
            // among siblings the order of D is the order of (count, then token).  Their places
            // follow from one pass per distinct count, largest first, without any merging.
            double dc = 0.0;
            if (pass) {
                dc = __dmul_rn(d_parent, __ddiv_rn((double)e.y, dsum));      // Eq. 2 with Eq. 1
                if ((unsigned)e.w & RUN_COUNT_MASK) prefetch_l2(ent + e.z);   // likely looked at soon
            }
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
        // The children of this chunk are offered best first: (count, then smaller token) orders
        // siblings like their D values, and the first one that does not enter ends the chunk.
        unsigned rem = __ballot_sync(FULL, pass);
        while (rem) {
            const bool in = (rem >> lane) & 1u;
            const unsigned top = __reduce_max_sync(FULL, in ? (unsigned)e.y : 0u);
            const int src = __ffs(__ballot_sync(FULL, in && (unsigned)e.y == top)) - 1;    // smallest token among them
            const double dc = __dmul_rn(d_parent, __ddiv_rn((double)top, dsum));          // Eq. 2 with Eq. 1
            const int cz = __shfl_sync(FULL, e.z, src);
            const unsigned cw = (unsigned)__shfl_sync(FULL, e.w, src);
            if (!frontier_insert(F, fh, fs, K, dc, __shfl_sync(FULL, e.x, src), par_index, cz, cw, lane)) break;
            if (lane == 0 && (cw & RUN_COUNT_MASK)) prefetch_l2(ent + cz);                 // likely looked at soon
            rem &= ~(1u << src);
        }
    }
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
                // With a full frontier a child only matters if it beats the worst entry.  Counts are
                // at least 1, so the sibling sum is at least cur_n and D <= cur_d * count / cur_n:
                // children below the count that needs are skipped without any arithmetic.
                int cmin = 1;
                if (fs == K) {
                    const double need = W.F.d[(fh + fs - 1) & (SD_MAX_SPEC - 1)] / cur_d * (double)cur_n * 0.999999;
                    cmin = need >= 2.0e9 ? 2000000000 : max(1, (int)need);
                }
                int ts;
                scan_run_by_count(ent, cur_cb, cur_n, 0, 1, cur_idx, cmin, W, W.T, 0, ts, K, sum, lane);
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

// MatchPattern in the global tree, from a node that is already known: descends tx[from .. to).
// Levels whose child run lies inside the window already in registers cost no memory access.
// Returns the node reached (-1: no match), its child run (cb, wfull) and its COUNT.
__device__ int walk_from(const int4* __restrict__ ent, int limit, int node, const int* tx, int from, int to, int lane,
                         int& cb, unsigned& wfull, int& count) {
    if (node < 0) return -1;
    int wb = node;
    int4 w = load_window(ent, wb, limit, lane);
    cb = __shfl_sync(FULL, w.z, 0);
    wfull = (unsigned)__shfl_sync(FULL, w.w, 0);
    count = __shfl_sync(FULL, w.y, 0);
    int n = (int)(wfull & RUN_COUNT_MASK);
    for (int pos = from; pos < to; ++pos) {
        const int x = tx[pos];
        if (n == 0) return -1;
        if (n > 32) {                                           // wide run: 32-way search
            int4 e;
            node = find_child_entry(ent, cb, n, x, lane, e);
            if (node < 0) return -1;
            cb = e.z; wfull = (unsigned)e.w; count = e.y; n = (int)(wfull & RUN_COUNT_MASK);
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
        count = __shfl_sync(FULL, w.y, src);
        n = (int)(wfull & RUN_COUNT_MASK);
    }
    return node;
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

// ---------------------------------------------------------------------------------------------
// A job whose match node has more than 32 occurrences, over a list of occurrences that is SORTED
// by the text behind them.  Every node below the match node is a range of the list (the items
// that agree on the tokens so far), its children are the runs of equal next tokens inside the
// range, and expanding a node is one pass over its own range.
//   Per-request tree: the list is the suffix order of the request's text (suffix_order.cuh), the
//   pattern's occurrences are the range S[lo .. hi), COUNT is the size of a range.
//   Global tree: the list is the base node's range of the offline build's suffix order, staged
//   with the tokens around every occurrence; the job of pattern length p counts only the items
//   that match at least p tokens (FILTER).
// Frontier: the sorted ring of the tree-entry path; fields cb / nc hold the candidate's range as
// lo / (hi << 5 | depth below the match node).
struct TextItems {            // items j of S: suffixes that start with the pattern of length p
    const int* tx; const int* S; int t, p;
    // token `level` (1: the first one behind the pattern) of item j, -1 if the text ends before it
    __device__ __forceinline__ int tok(int j, int level) const { const int q = S[j] + p - 1 + level; return q <= t - 1 ? tx[q] : -1; }
    __device__ __forceinline__ bool member(int) const { return true; }
};
struct WindowItems {          // items j: occurrences of the global base pattern, with 64 tokens around each
    const int (*gwin)[64]; const int* avail; const int* ell; int base_p, p;
    __device__ __forceinline__ int tok(int j, int level) const { return level <= avail[j] ? gwin[j][31 + base_p + level] : -1; }
    __device__ __forceinline__ bool member(int j) const { return ell[j] >= p; }
};

template <bool FILTER, class Items, class BlockShared>
__device__ void expand_range(BlockShared& sh, WarpWork& W, const Items& it, int lo0, int hi0, int tree, int p, int budget,
                             int dlim, unsigned flags, int lane) {
    const int order = tree * SD_MAX_DEPTH + p;
    const int buf = W.best_buf ^ 1;
    Frontier& F = W.F;
    int fh = 0, fs = 0, cnt = 0;
    double score = 0.0;
    bool dropped = false;
    double cur_d = 1.0;
    int lo = lo0, hi = hi0, cur_k = 0, cur_idx = -1;
    bool have_cur = true;
    while (true) {
        if (!have_cur) {
            if (cnt >= budget || fs == 0) break;
            cur_d = F.d[fh];
            const int tok = F.tok[fh], par = F.par[fh];
            lo = F.cb[fh];
            hi = (int)(F.nc[fh] >> 5);
            cur_k = (int)(F.nc[fh] & 31u);
            if ((score + (double)(budget - cnt) * cur_d) * 1.000000001 < best_so_far(sh)) { dropped = true; break; }
            __syncwarp();
            fh = (fh + 1) & (SD_MAX_SPEC - 1);
            --fs;
            if (lane == 0) { W.tok[buf][cnt] = tok; W.par[buf][cnt] = (unsigned char)(par + 1); }
            score = __dadd_rn(score, cur_d);                    // Eq. 4, insertion order
            if (lane == 0) atomicMax(&sh.best_hi, (unsigned)__double2hiint(score));
            cur_idx = cnt++;
            const int K = budget - cnt;
            if (fs > K) fs = K;
            if (flags & SD_FLAG_LINEAR) fs = 0;
        }
        have_cur = false;
        if (cnt >= budget) break;
        if (cur_k >= dlim || lo >= hi) continue;                // depth cap: the node has no children
        const int K = budget - cnt;
        const int level = cur_k + 1;
        // the sibling sum (denominator of Eq. 1): items of the job that have a next token
        int sum;
        if (FILTER) {
            sum = 0;
            for (int base = lo; base < hi; base += 32) {
                const int j = base + lane;
                sum += __popc(__ballot_sync(FULL, j < hi && it.member(j) && it.tok(j, level) >= 0));
            }
        } else {
            sum = hi - lo - (it.tok(lo, level) < 0 ? 1 : 0);    // an item whose text ends here sorts first; all others go on
        }
        if (sum <= 0) continue;
        const double dsum = (double)sum;
        // the runs of equal next tokens; an open run is carried from chunk to chunk
        int run_tok = -2, run_lo = lo, run_c = 0;               // -2: none yet
        for (int base = lo; base < hi + 32; base += 32) {       // (a last round behind the range closes the last run)
            const int j = base + lane;
            int tk = -3;                                        // behind the range: differs from every token
            bool mem = false;
            if (j < hi) { tk = it.tok(j, level); mem = FILTER ? (tk >= 0 && it.member(j)) : true; }
            int prev = __shfl_up_sync(FULL, tk, 1);
            if (lane == 0) prev = run_tok;
            const bool bnd = tk != prev;                        // a run starts here
            const unsigned bm = __ballot_sync(FULL, bnd);
            const unsigned mm = FILTER ? __ballot_sync(FULL, mem) : 0u;
            if (!bm) { if (FILTER) run_c += __popc(mm); }
            else {
                // every boundary closes the run that ends right before it: the open run for the
                // first boundary of the chunk, else the run that began at the boundary before
                const unsigned lt = (1u << lane) - 1u;
                const unsigned below = bm & lt;
                const int sb = below ? 31 - __clz(below) : 0;
                const int s_tok = __shfl_sync(FULL, tk, sb);
                const int c_tok = below ? s_tok : run_tok, c_lo = below ? base + sb : run_lo, c_hi = base + lane;
                int c_cnt = c_hi - c_lo;
                if (FILTER) c_cnt = below ? __popc(mm & lt & ~((1u << sb) - 1u)) : run_c + __popc(mm & lt);
                bool pass = bnd && c_tok >= 0 && c_cnt > 0;
                double dc = 0.0;
                if (pass) {
                    dc = __dmul_rn(cur_d, __ddiv_rn((double)c_cnt, dsum));             // Eq. 2 with Eq. 1
                    if (fs == K) {
                        const int last = (fh + fs - 1) & (SD_MAX_SPEC - 1);
                        pass = better(dc, c_tok, cur_idx, F.d[last], F.tok[last], F.par[last]);
                    }
                }
                unsigned pm = __ballot_sync(FULL, pass);
                while (pm) {
                    const int src = __ffs(pm) - 1;
                    pm &= pm - 1;
                    frontier_insert(F, fh, fs, K, __shfl_sync(FULL, dc, src), __shfl_sync(FULL, c_tok, src), cur_idx,
                                    __shfl_sync(FULL, c_lo, src),
                                    ((unsigned)__shfl_sync(FULL, c_hi, src) << 5) | (unsigned)level, lane);
                }
                const int lb = 31 - __clz(bm);                  // the last boundary opens the run that is carried on
                run_tok = __shfl_sync(FULL, tk, lb);
                run_lo = base + lb;
                if (FILTER) run_c = __popc(mm & ~((1u << lb) - 1u));
            }
            if (base >= hi) break;
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

struct StepArgs {             // what one launch needs beyond the store
    int n;
    const int32_t* d_slot;
    int Pe;
    double alpha;
    int max_spec;
    unsigned flags;
    double tau;
    const int32_t* d_budget_cap;
    int32_t *d_n_draft, *d_tokens, *d_parents, *d_positions;
    uint32_t* d_mask;
    int32_t *d_chosen_tree, *d_chosen_p;
    double* d_score;
    int32_t* d_status;
    const int64_t* d_app_off;     // sd_step: the tokens to append first (NULL: sd_speculate)
    const int32_t* d_app_tok;
    int stage_tokens;             // tokens of text, and entries of its suffix order, the block can hold in shared
                                  // memory (0: the text is too long; both are then used in place)
    int32_t* scratch;             // [n][Tp] by request: the suffix order of a text that is not staged
};

template <int WARPS, int MINB>
__global__ void __launch_bounds__(WARPS * 32, MINB) speculate_fused_kernel(sd_store sv, StepArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    using BlockShared = BlockSharedT<WARPS>;
    constexpr int NT = WARPS * 32;
    BlockShared& sh = *reinterpret_cast<BlockShared*>(smem_raw);
    int* const stx = reinterpret_cast<int*>(smem_raw + ((sizeof(BlockShared) + 15) & ~(size_t)15));
    const int tid = threadIdx.x, lane = tid & 31, wib = tid >> 5;
    const int i = blockIdx.x;
    const int M = sv.M, words = (M + 31) / 32, D = sv.D, Pe = a.Pe;
    const unsigned flags = a.flags;
    const int slot = a.d_slot[i];
    const bool ok = slot >= 0 && slot < sv.R;
    int t = 0, status = SD_STATUS_BAD_SLOT, sa_buf = 0;
    SlotState* ss = nullptr;
    int32_t* gtext = nullptr;
    if (ok) {
        ss = sv.s_state + slot; t = ss->len; status = ss->status; sa_buf = ss->sa_buf;
        gtext = sv.s_text + (long long)slot * sv.Tp;
    }
    const int t_old = t;
    if (tid < 2 * SD_MAX_DEPTH) { (&sh.node[0][0])[tid] = -1; (&sh.nc[0][0])[tid] = 0; }
    if (tid < SD_MAX_DEPTH + 2) sh.g_cum[tid] = 0;
    if (tid <= SD_MAX_DEPTH) { sh.r_lo[tid] = 0; sh.r_cnt[tid] = 0; }
    if (tid < SD_MAX_DEPTH) { sh.g_cnt[tid] = 0; sh.g_rank[tid] = -1; }
    if (tid == 0) {
        sh.njobs = 0; sh.next = 0; sh.nwide = 0; sh.nwide_kept = 0; sh.best_hi = 0u; sh.win_warp = -1;
        sh.first_bad = 0x7fffffff;
        sh.g_walked = 0; sh.g_failed = 0; sh.g_base_p = 0; sh.g_base_m = 0;
    }
    WarpWork& W = sh.w[wib];
    if (lane == 0) { W.best_score = 0.0; W.best_order = 1 << 30; W.best_n = 0; W.best_buf = 0; }
    __syncthreads();

    // ---------------- 0. sd_step: the accepted tokens go behind the request's text
    const int32_t* newtok = nullptr;
    int take = 0;
    if (a.d_app_off && ok) {
        const long long b0 = a.d_app_off[i];
        const int n_new = (int)(a.d_app_off[i + 1] - b0);
        newtok = a.d_app_tok + b0;
        if (n_new > 0 && !(status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN))) {
            take = min(n_new, sv.T - t_old);
            for (int k = tid; k < take; k += NT) {
                const int x = newtok[k];
                if (x < 0 || x >= sv.V) atomicMin(&sh.first_bad, k);
            }
            __syncthreads();
            const int good = min(take, sh.first_bad);
            if (good < take) status |= SD_STATUS_BAD_TOKEN;     // the text stops before the first bad token
            else if (take < n_new) status |= SD_STATUS_POOL_FULL;
            take = good;
            for (int k = tid; k < take; k += NT) gtext[t_old + k] = newtok[k];
            t = t_old + take;
        }
    }
    const bool usable = ok && !(status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN)) && t > 0;
    int cap = a.max_spec;
    if (a.d_budget_cap && a.d_budget_cap[i] >= 0) cap = min(cap, a.d_budget_cap[i]);
    const bool want_g = usable && !(flags & SD_FLAG_REQUEST_ONLY);
    const bool want_r = usable && !(flags & SD_FLAG_GLOBAL_ONLY);

    // ---------------- 1. the text and its suffix order
    const bool staged = t <= a.stage_tokens;
    int fin_a0 = -1;
    const int* tx = stx;
    int* S = stx + a.stage_tokens;
    if (ok && (usable || take > 0)) {
        if (staged) {
            const int4* g4 = reinterpret_cast<const int4*>(gtext);
            int4* s4 = reinterpret_cast<int4*>(stx);
            for (int g = tid; g * 4 < t; g += NT) {
                int4 v = make_int4(0, 0, 0, 0);
                if (g * 4 < t_old) v = g4[g];
                // (the new tokens come from the call's list: the copy in the text buffer above may not have landed yet)
                int* c = reinterpret_cast<int*>(&v);
#pragma unroll
                for (int u = 0; u < 4; ++u) { const int q = g * 4 + u; if (q >= t_old && q < t) c[u] = newtok[q - t_old]; }
                s4[g] = v;
            }
        } else {
            tx = gtext;                                         // too long to stage: text and order are used in place
            S = a.scratch + (long long)i * sv.Tp;
        }
        int32_t* sa[2] = {sv.s_sa + (long long)slot * sv.Tp, sv.s_sa + ((long long)sv.R + slot) * sv.Tp};
        if (staged || take > 0)
            for (int k = tid; k < t_old; k += NT) S[k] = sa[sa_buf][k];
        else
            S = sa[sa_buf];                                     // nothing to merge: the stored order is read as it is
        __syncthreads();                                        // (also: the new tokens in gtext are visible to the block)
        for (int t0 = t_old; t0 < t; t0 += SA_CHUNK) {
            sa_merge_chunk<NT>(tx, t0, min(t, t0 + SA_CHUNK), D, S, sa[sa_buf], sa[sa_buf ^ 1], sh.sat, tid);
            sa_buf ^= 1;
            fin_a0 = max(0, t0 - (D - 1));                      // sh.sat.fin[a - fin_a0]: where the last merge put suffix a
        }
        if (tid == 0 && take > 0) { ss->len = t; ss->sa_buf = sa_buf; }
    }
    if (tid == 0 && ok && a.d_app_off) ss->status = status;
    __syncthreads();

    // ---------------- 2. match
    if (wib == 0) {
        // the slot's cached global match nodes (taken at context length g_len <= t)
        int depths = 0, kk = 0;
        if (usable) {
            const bool cache_ok = ss->g_gen == ss->gen && ss->g_epoch == sv.g_state->epoch && ss->g_len <= t && ss->g_len > 0;
            if (cache_ok) { depths = ss->g_depths; kk = t - ss->g_len; }
            sh.g_src[lane] = (cache_ok && lane < depths) ? ss->g_node[lane] : -1;
        }
        if (lane == 0) { sh.g_src_depths = depths; sh.g_src_k = kk; }
    }
    __syncthreads();
    const int Lcap = min(Pe, D - 1);                            // a match node at depth D has no children
    // Per-request tree: the range of every pattern in the suffix order, a warp per pattern length.
    // Its first suffix is the context's own end (the pattern followed by nothing); the earlier
    // occurrences follow it.
    const int Lr = want_r ? min(Lcap, t - 1) : 0;
    auto request_ranges = [&]() {
        for (int p = wib + 1; p <= Lr; p += WARPS) {
            // the range begins with the context's own end, whose place the merge above may have just found
            const int lo = fin_a0 >= 0 ? sh.sat.fin[t - p - fin_a0] : pattern_lo_warp(tx, t, S, t - p, p, lane);
            const int hi = pattern_hi_warp(tx, t, S, t - p, p, lo, lane);
            if (lane == 0) { sh.r_lo[p] = lo; sh.r_cnt[p] = max(hi - lo - 1, 0); }
        }
    };
    // Global tree: rounds of WARPS pattern lengths, shortest first, until a node can serve as
    // the base of occurrence mode, a pattern does not occur, or all lengths are done.
    const int PeG = want_g ? min(Pe, t) : 0;
    const bool occ_mode = sv.g_lo != nullptr;
    for (int r0 = 0; r0 < PeG; r0 += WARPS) {
        const int p = r0 + wib + 1;
        if (p <= PeG) {
            int cb = 0, cntn = 0;
            unsigned wf = 0;
            // from the cached node of the tokens before the new ones, if there is one; else from the root table
            const int kk = sh.g_src_k;
            int node, from;
            if (p > kk && p - kk <= sh.g_src_depths) { node = sh.g_src[p - kk - 1]; from = t - kk; }
            else { const int x0 = tx[t - p]; node = (x0 >= 0 && x0 < sv.V) ? sv.g_root[x0] : -1; from = t - p + 1; }
            node = walk_from(sv.g_ent, (int)sv.g_cap, node, tx, from, t, lane, cb, wf, cntn);
            int rank = -1;
            const int nch = (int)(wf & RUN_COUNT_MASK);
            // usable as base: at most 64 occurrences, laid down by the offline build, never touched since
            const bool elig = occ_mode && node >= 0 && cntn <= SD_OCC_BASE && !(wf & NODE_TOUCHED) &&
                              (nch == 0 || ((wf & RUN_STATIC) && cb < sv.static_entries));
            if (elig && nch > 0 && lane == 0) rank = sv.g_lo[cb];
            if (lane == 0) {
                sh.node[0][p - 1] = node;
                if (node >= 0) { sh.cb[0][p - 1] = cb; sh.nc[0][p - 1] = wf; sh.g_cnt[p - 1] = cntn; }
                else atomicOr(&sh.g_failed, 1);
                sh.g_rank[p - 1] = elig ? (nch > 0 ? rank : -2) : -1;   // -2: usable, and known to have no children
            }
        }
        if (r0 == 0) request_ranges();
        __syncthreads();
        if (tid == 0) {
            const int hi = min(PeG, r0 + WARPS);
            sh.g_walked = hi;
            for (int p = r0 + 1; p <= hi && sh.g_base_p == 0; ++p)
                if (sh.node[0][p - 1] >= 0 && sh.g_rank[p - 1] != -1) sh.g_base_p = p;
        }
        __syncthreads();
        if (sh.g_base_p || sh.g_failed) break;
    }
    if (PeG == 0) request_ranges();
    __syncthreads();
    if (wib == 0 && PeG > 0) {
        // the match nodes of this context, for the next call.  A pattern that does not occur ends
        // the list: no longer one occurs either.
        const int walked = sh.g_walked, failed = sh.g_failed;
        const int depths = failed ? SD_MAX_DEPTH : walked;
        if (lane < depths) ss->g_node[lane] = lane < walked ? sh.node[0][lane] : -1;
        if (lane == 0) { ss->g_gen = ss->gen; ss->g_epoch = sv.g_state->epoch; ss->g_len = t; ss->g_depths = depths; }
    }
    // the base's occurrences (first pattern token, suffix length)
    const int base_p = sh.g_base_p;
    if (wib == 1 && base_p > 0) {
        const int rank = sh.g_rank[base_p - 1];
        const int m = rank >= 0 ? sh.g_cnt[base_p - 1] : 0;
        for (int o = lane; o < m; o += 32) {
            const int pos = (int)sv.g_sa[rank + o];
            sh.g_pos[o] = pos;
            sh.g_avail[o] = (int)sv.g_len[rank + o] - base_p;
            sh.g_ell[o] = (int)sv.g_back[pos];                  // for now: tokens before the occurrence in its sequence
        }
        if (lane == 0) sh.g_base_m = m;
    }
    __syncthreads();
    const int base_m = sh.g_base_m;
    // the 64 tokens around every occurrence of the base (one coalesced row per occurrence)
    for (int o = wib; o < base_m; o += WARPS) {
        const long long pos = sh.g_pos[o];
        const long long q0 = pos - 32 + lane, q1 = pos + lane;
        sh.gwin[o][lane] = (q0 >= 0) ? sv.g_text[q0] : -1;
        sh.gwin[o][32 + lane] = (q1 < sv.N0) ? sv.g_text[q1] : -1;
    }
    __syncthreads();
    if (wib == 0 && base_m > 0) {
        // how far back every occurrence of the base agrees with the context
        int ell[SD_OCC_BASE / 32];
#pragma unroll
        for (int u = 0; u < SD_OCC_BASE / 32; ++u) {
            const int o = lane + 32 * u;
            ell[u] = 0;
            if (o < base_m) {
                const int back = sh.g_ell[o];
                const int lim = min(Lcap, t);
                int l = base_p;
                while (l < lim && l - base_p < back && sh.gwin[o][31 - (l - base_p)] == tx[t - 1 - l]) ++l;
                sh.g_ell[o] = l;
                ell[u] = l;
            }
        }
        // lane L: occurrences that match at least L + 1 tokens
        int c = 0;
#pragma unroll
        for (int u = 0; u < SD_OCC_BASE / 32; ++u)
            for (int o = 0; o < 32; ++o) c += (__shfl_sync(FULL, ell[u], o) >= lane + 1) ? 1 : 0;
        sh.g_cum[lane + 1] = lane + 1 >= base_p ? c : 0;
    }
    __syncthreads();

    // ---------------- 3. job queue, costliest first; tree-entry jobs that start at a wide node wait
    if (tid < 2 * SD_MAX_DEPTH) {
        const int tree = tid / SD_MAX_DEPTH, p = tid % SD_MAX_DEPTH + 1;
        int c = 0;
        if (p <= Pe && p <= Lcap) {
            bool has = false;
            if (tree == 1) has = p <= Lr && sh.r_cnt[p] > 0;
            else if (base_p > 0 && p >= base_p) has = sh.g_cum[p] > 0;
            else if (p <= sh.g_walked) {
                const unsigned wf = sh.nc[0][p - 1];
                const int nch = (int)(wf & RUN_COUNT_MASK);
                has = sh.node[0][p - 1] >= 0 && nch > 0;
                if (has) {
                    // all first runs start their way to L2 now, long before a warp gets to them
                    const int4* base = sv.g_ent + sh.cb[0][p - 1];
                    const int lines = min(4, (nch + 7) >> 3);
                    for (int l = 0; l < lines; ++l) prefetch_l2(base + l * 8);
                }
            }
            if (has) {
                c = min(budget_for(a.alpha, p, cap), D - p);      // an upper bound of the job's SCORE, see below
                if (c > 0 && tree == 0 && !(base_p > 0 && p >= base_p)) {
                    const unsigned wf = sh.nc[0][p - 1];
                    if ((int)(wf & RUN_COUNT_MASK) > WIDE_RUN && !(wf & RUN_HAS_TOP)) { sh.wide[atomicAdd(&sh.nwide, 1)] = tid; c = 0; }
                }
            }
        }
        sh.cost[tid] = c;
    }
    __syncthreads();
    if (tid < 2 * SD_MAX_DEPTH) {
        const int c = sh.cost[tid];
        if (c > 0) {
            int rank = 0;
            for (int q = 0; q < 2 * SD_MAX_DEPTH; ++q) {
                const int cq = sh.cost[q];
                rank += (cq > c || (cq == c && q < tid)) ? 1 : 0;
            }
            sh.job[rank] = tid;
            atomicAdd(&sh.njobs, 1);
        }
    }
    __syncthreads();
    const int njobs = sh.njobs;
    while (true) {
        int j = 0;
        if (lane == 0) j = atomicAdd(&sh.next, 1);
        j = __shfl_sync(FULL, j, 0);
        if (j >= njobs) break;
        const int code = sh.job[j];
        const int tree = code / SD_MAX_DEPTH, p = code % SD_MAX_DEPTH + 1;
        const int budget = budget_for(a.alpha, p, cap);
        // SCORE <= number of draft nodes (every D <= 1), and SCORE <= number of levels below the
        // match node: the D values of one level of a tree add up to at most 1 (Eq. 1 shares out the
        // parent's D among its children).  A job that cannot reach the best score so far is skipped.
        if ((double)min(budget, D - p) * 1.000000001 < best_so_far(sh)) continue;
        if (tree == 1) {
            const int m = sh.r_cnt[p], lo = sh.r_lo[p] + 1;
            if (m <= SD_OCC_LANES) {
                const int e = lane < m ? S[lo + lane] + p - 1 : 0;       // the occurrence's last pattern token
                const int kmax = lane < m ? min(t - 1 - e, D - p) : 0;
                expand_occ(sh, W, tx + e, kmax, 1, p, budget, flags, lane);
            } else {
                expand_range<false>(sh, W, TextItems{tx, S, t, p}, lo, lo + m, 1, p, budget, D - p, flags, lane);
            }
        } else if (base_p > 0 && p >= base_p) {
            if (sh.g_cum[p] <= SD_OCC_LANES) {
                // a lane per occurrence that matches p tokens: lane i takes the i-th of them
                unsigned mk[SD_OCC_BASE / 32];
                int o = -1, left = lane + 1;
#pragma unroll
                for (int u = 0; u < SD_OCC_BASE / 32; ++u) {
                    mk[u] = __ballot_sync(FULL, lane + 32 * u < base_m && sh.g_ell[lane + 32 * u] >= p);
                    const int c = __popc(mk[u]);
                    if (o < 0 && left <= c) o = 32 * u + (int)__fns(mk[u], 0, left);
                    left -= c;
                }
                const int kmax = o >= 0 ? min(sh.g_avail[o], D - p) : 0;
                expand_occ(sh, W, &sh.gwin[o >= 0 ? o : 0][31 + base_p], kmax, 0, p, budget, flags, lane);
            } else {
                expand_range<true>(sh, W, WindowItems{sh.gwin, sh.g_avail, sh.g_ell, base_p, p}, 0, base_m, 0, p, budget, D - p,
                                   flags, lane);
            }
        } else {
            expand_job(sh, W, sv.g_ent, (int)sv.g_cap, 0, p, budget, flags, false, 0, lane);
        }
    }
    __syncthreads();
    // Tree-entry jobs that start at a wide node (short patterns, hence small budgets): most cannot
    // reach the best score any more and are dropped here.  For the rest the warps of the block share
    // the scan of the run, then one warp merges the partial lists and finishes the job.
    if (tid == 0) {
        const double best = __hiloint2double((int)sh.best_hi, 0);
        int kept = 0;
        for (int q = 0; q < sh.nwide; ++q) {
            const int p = sh.wide[q] % SD_MAX_DEPTH + 1;
            if (!((double)min(budget_for(a.alpha, p, cap), D - p) * 1.000000001 < best)) sh.wide[kept++] = sh.wide[q];
        }
        sh.nwide_kept = kept;
    }
    __syncthreads();
    const int nwide = sh.nwide_kept;
    for (int base = 0; base < nwide; base += WARPS) {
        const int nj = min(WARPS, nwide - base);
        const int G = WARPS / nj;                               // warps per job
        const int my_job = wib / G, my_slice = wib % G;
        const bool active = my_job < nj;
        int p = 1, budget = 0, fs = 0;
        if (active) {
            const int code = sh.wide[base + my_job];
            p = code % SD_MAX_DEPTH + 1;
            budget = budget_for(a.alpha, p, cap);
            long long sum;
            scan_run_by_count(sv.g_ent, sh.cb[0][p - 1], (int)(sh.nc[0][p - 1] & RUN_COUNT_MASK), my_slice, G, -1, 1, W,
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
            expand_job(sh, W, sv.g_ent, (int)sv.g_cap, 0, p, budget, flags, true, fs, lane);
        }
        __syncthreads();
    }

    // ---------------- 4. select (first in loop order among the largest scores) and emit
    if (wib == 0) {
        double sc = lane < WARPS ? sh.w[lane].best_score : 0.0;
        int od = lane < WARPS ? sh.w[lane].best_order : 1 << 30;
        int ww = lane;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const double osc = __shfl_xor_sync(FULL, sc, off);
            const int ood = __shfl_xor_sync(FULL, od, off);
            const int oww = __shfl_xor_sync(FULL, ww, off);
            if (osc > sc || (osc == sc && ood < od)) { sc = osc; od = ood; ww = oww; }
        }
        // Section 3.2: the tree is used only if its score exceeds the threshold (tau = 0: any score above 0)
        if (lane == 0) sh.win_warp = (sc > 0.0 && sc > a.tau) ? ww : -1;
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
            for (int an = j, hops = 0; an >= 0 && hops < SD_MAX_SPEC; an = (int)wpar[an] - 1, ++hops) {
                bits |= 1ull << an;
                ++depth;
            }
            pos = t + depth - 1;
        }
        const long long o = (long long)i * M + j;
        a.d_tokens[o] = tok; a.d_parents[o] = par; a.d_positions[o] = pos;
        a.d_mask[o * words] = (uint32_t)bits;
        if (words > 1) a.d_mask[o * words + 1] = (uint32_t)(bits >> 32);
    }
    if (tid == 0) {
        a.d_n_draft[i] = nd; a.d_chosen_tree[i] = ctree; a.d_chosen_p[i] = cp; a.d_score[i] = best;
        if (a.d_status) a.d_status[i] = status;
    }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// Launch.  Block shapes (measured): two blocks per SM is the usual one; a batch of at most one
// request per SM gets bigger blocks, a batch of more than two requests per SM smaller ones
// (four per SM) to stay in one wave.  The text of a request is staged in shared memory when it
// fits beside the block's working set, else it is read in place.
namespace {

constexpr int CTA_WARPS = 10;
constexpr int CTA_WARPS_WIDE = 16;
constexpr int CTA_WARPS_NARROW = 5;
constexpr int SMEM_PER_SM = 228 * 1024;       // shared memory of one SM; a block also costs 1 KB of it
constexpr int MAX_DEVICES = 64;

struct DeviceInfo {
    bool ready = false;
    int sm_count = 0;
};
DeviceInfo g_dev[MAX_DEVICES];
std::mutex g_dev_mutex;

template <int WARPS, int MINB>
constexpr int stage_limit_tokens() {
    return (int)((SMEM_PER_SM / MINB - 1024 - (int)((sizeof(BlockSharedT<WARPS>) + 15) & ~(size_t)15)) / 4) & ~3;
}

// once per device: raise the kernels' dynamic shared memory limit, read the SM count
int device_setup(int dev, int* sm_count) {
    if (dev < 0 || dev >= MAX_DEVICES) return SD_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_dev[dev].ready) {
        SD_CUDA_OK(cudaFuncSetAttribute(speculate_fused_kernel<CTA_WARPS, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        SMEM_PER_SM / 2 - 1024));
        SD_CUDA_OK(cudaFuncSetAttribute(speculate_fused_kernel<CTA_WARPS_WIDE, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        SMEM_PER_SM - 1024));
        SD_CUDA_OK(cudaFuncSetAttribute(speculate_fused_kernel<CTA_WARPS_NARROW, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        SMEM_PER_SM / 4 - 1024));
        SD_CUDA_OK(cudaDeviceGetAttribute(&g_dev[dev].sm_count, cudaDevAttrMultiProcessorCount, dev));
        g_dev[dev].ready = true;
    }
    *sm_count = g_dev[dev].sm_count;
    return SD_OK;
}

template <int WARPS, int MINB>
void launch_shape(const sd_store& s, StepArgs a, cudaStream_t st) {
    // shared memory behind the block's working set: the text and its suffix order (as many entries), if they fit
    const int lim = stage_limit_tokens<WARPS, MINB>();
    a.stage_tokens = 2 * s.Tp <= lim ? s.Tp : 0;
    const size_t smem = ((sizeof(BlockSharedT<WARPS>) + 15) & ~(size_t)15) + (size_t)a.stage_tokens * 8;
    speculate_fused_kernel<WARPS, MINB><<<(unsigned)a.n, WARPS * 32, smem, st>>>(s, a);
}

int launch_fused(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm, const int32_t* d_budget_cap,
                 int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask,
                 int32_t* d_chosen_tree, int32_t* d_chosen_p, double* d_score, int32_t* d_status,
                 const int64_t* d_app_off, const int32_t* d_app_tok, bool step, int32_t* scratch, void* stream) {
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
    int sms = 0;
    const int rc = device_setup(s->device, &sms);
    if (rc != SD_OK) return rc;
    StepArgs a;
    a.n = n; a.d_slot = d_slot;
    a.Pe = prm->P < s->D ? prm->P : s->D;                       // longer patterns never match
    a.alpha = prm->alpha; a.max_spec = prm->max_spec; a.flags = prm->flags; a.tau = prm->tau;
    a.d_budget_cap = d_budget_cap;
    a.d_n_draft = d_n_draft; a.d_tokens = d_tokens; a.d_parents = d_parents; a.d_positions = d_positions;
    a.d_mask = d_mask; a.d_chosen_tree = d_chosen_tree; a.d_chosen_p = d_chosen_p; a.d_score = d_score;
    a.d_status = d_status;
    a.d_app_off = step ? d_app_off : nullptr; a.d_app_tok = step ? d_app_tok : nullptr;
    a.stage_tokens = 0;
    a.scratch = scratch;
    cudaStream_t st = (cudaStream_t)stream;
    // a text too long for the usual shape's shared memory may still fit the one-block-per-SM shape
    const bool long_text = 2 * s->Tp > stage_limit_tokens<CTA_WARPS, 2>();
    if (n <= sms || (long_text && n <= 2 * sms)) launch_shape<CTA_WARPS_WIDE, 1>(*s, a, st);
    else if (n > 2 * sms && 2 * s->Tp <= stage_limit_tokens<CTA_WARPS_NARROW, 4>()) launch_shape<CTA_WARPS_NARROW, 4>(*s, a, st);
    else launch_shape<CTA_WARPS, 2>(*s, a, st);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}

}  // namespace

extern "C" int sd_speculate(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm,
                            const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents,
                            int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
                            double* d_score, int32_t* d_status, void* stream) {
    return launch_fused(s, n, d_slot, prm, d_budget_cap, d_n_draft, d_tokens, d_parents, d_positions, d_mask, d_chosen_tree,
                        d_chosen_p, d_score, d_status, nullptr, nullptr, false, s ? s->occ_scratch : nullptr, stream);
}

extern "C" int sd_step(sd_store* s, int32_t n, const int32_t* d_slot, const int64_t* d_offsets, const int32_t* d_new_tokens,
                       const sd_spec_params* prm, const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens,
                       int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree,
                       int32_t* d_chosen_p, double* d_score, int32_t* d_status, void* stream) {
    return launch_fused(s, n, d_slot, prm, d_budget_cap, d_n_draft, d_tokens, d_parents, d_positions, d_mask, d_chosen_tree,
                        d_chosen_p, d_score, d_status, d_offsets, d_new_tokens, true, s ? s->occ_scratch : nullptr, stream);
}

// ---------------------------------------------------------------------------------------------
// sd_speculate_noalloc: sd_speculate with the kernel's scratch memory (the occurrence lists that
// do not fit shared memory) in a fixed array that is part of the loaded library image instead of
// in memory the store obtained from cudaMalloc.  Meant for callers that must not touch the CUDA
// allocator at all (see the declaration in suffixspec.h).
//
// The array's name below is only meaningful to device code.  Host code holds a stand-in
// symbol of the same name, so the launch code first asks the runtime for the array's
// real device address (once per device, with that device current) and passes that on.
namespace {

static __device__ __align__(256) int32_t g_noalloc_scratch[SD_NOALLOC_MAX_TOKENS];

int32_t* g_noalloc_ptr[MAX_DEVICES];          // device address of the array, per device
bool g_noalloc_ready[MAX_DEVICES];
std::mutex g_noalloc_mutex;

// Device address of the scratch array on the current device (looked up on first use).
int noalloc_scratch_address(int32_t** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return SD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ready[dev]) {
        int32_t* p = nullptr;
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
    if (!s || n < 0 || n > s->R) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    // one row of max_req_tokens (rounded up to 4) per request: the batch must fit the fixed array
    if ((long long)n * s->Tp > SD_NOALLOC_MAX_TOKENS) return SD_ERR_CAPACITY;
    int32_t* base = nullptr;
    const int rc = noalloc_scratch_address(&base);
    if (rc != SD_OK) return rc;
    // Every list the kernel reads from the array was written by the same block earlier in the same
    // launch, so nothing left over from an earlier call is ever consumed and nothing needs clearing.
    return launch_fused(s, n, d_slot, prm, d_budget_cap, d_n_draft, d_tokens, d_parents, d_positions, d_mask, d_chosen_tree,
                        d_chosen_p, d_score, d_status, nullptr, nullptr, false, base, stream);
}
