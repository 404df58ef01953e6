// Suffix order of a request's text: how the implicit per-request tree is indexed.
//
// A per-request tree (Section 3: the tree over the request's prompt and generation so far) is
// kept as the text x_{1:t} plus the ORDER of its suffixes by their first D tokens (D = depth
// cap): sa[0 .. t) lists the start positions, smallest suffix first; a suffix that ends before
// another one's D-th token comes before its extensions, equal D-token strings go by position.
// In that order the occurrences of any string of at most D tokens are one contiguous range,
// sorted by the text that follows them: the range is the string's node, its size the node's
// COUNT, and the runs of equal next tokens inside it are the node's children.
//
// Appending tokens changes little of the order.  Only the suffixes that start less than D
// tokens before the old end (they grow) and the new ones need a place; everything else keeps
// its relative order.  sa_merge_chunk takes those (at most D - 1 + SA_CHUNK) suffixes out,
// finds the place of each among the kept ones by binary search, and writes the merged order.
#pragma once

#include "common.cuh"

namespace {

constexpr int SA_CHUNK = 64;                          // tokens appended per merge
constexpr int SA_MOVED = SA_CHUNK + SD_MAX_DEPTH;     // suffixes that get a new place in one merge

struct SaTemp {                                       // shared-memory scratch of one merge
    int rem[SD_MAX_DEPTH];                            // old indices of the entries that are taken out, ascending
    int rem_suf[SD_MAX_DEPTH];                        // the suffixes that sat there
    int n_rem;
    int r[SA_MOVED];                                  // per moved suffix: kept entries that come before it
    int fin[SA_MOVED];                                // its index in the merged order
    int rs[SA_MOVED];                                 // r, ascending
    int lmin[SA_MOVED];                               // tokens it shares with both kept neighbours (0: not known)
};

// Token i of the suffix that starts at s; -1 behind the end of the text (sorts before every token).
__device__ __forceinline__ int suf_tok(const int* tx, int t, int s, int i) { return s + i < t ? tx[s + i] : -1; }

// suffix a < suffix b ?  (whole warp; first D tokens, then position)
__device__ __forceinline__ bool suf_less_warp(const int* tx, int t, int D, int a, int b, int lane) {
    const int xa = lane < D ? suf_tok(tx, t, a, lane) : 0, xb = lane < D ? suf_tok(tx, t, b, lane) : 0;
    const unsigned diff = __ballot_sync(0xffffffffu, xa != xb);
    if (!diff) return a < b;
    const int f = __ffs(diff) - 1;
    return __shfl_sync(0xffffffffu, xa, f) < __shfl_sync(0xffffffffu, xb, f);
}

// the same by one thread
__device__ inline bool suf_less_thread(const int* tx, int t, int D, int a, int b) {
    for (int i = 0; i < D; ++i) {
        const int xa = suf_tok(tx, t, a, i), xb = suf_tok(tx, t, b, i);
        if (xa != xb) return xa < xb;
        if (xa < 0) break;                            // both end here (only possible for a == b)
    }
    return a < b;
}

// suffix a < suffix b, given that they agree on their first `from` tokens
__device__ inline bool suf_less_from(const int* tx, int t, int D, int a, int b, int from) {
    for (int i = from; i < D; ++i) {
        const int xa = suf_tok(tx, t, a, i), xb = suf_tok(tx, t, b, i);
        if (xa != xb) return xa < xb;
        if (xa < 0) break;
    }
    return a < b;
}

// The text grew from t0 to t1 tokens (t1 - t0 <= SA_CHUNK; tx holds all t1).  On entry S[0 .. t0)
// and g_old[0 .. t0) both hold the order for t0 tokens; on return S[0 .. t1) and g_new[0 .. t1)
// hold the order for t1 tokens (g_old and g_new are different arrays; S may be shared memory),
// and tmp.fin[a - a0] is the new index of every suffix a >= a0 = max(0, t0 - D + 1).
// All NT threads of the block call; ends with a barrier.
template <int NT>
__device__ void sa_merge_chunk(const int* tx, int t0, int t1, int D, int* S, const int* g_old, int* g_new, SaTemp& tmp,
                               int tid) {
    const int lane = tid & 31, wib = tid >> 5;
    constexpr int WARPS = NT / 32;
    const int a0 = max(0, t0 - (D - 1));                         // suffixes from here on grow or are new
    const int nA = t1 - a0;
    if (tid == 0) tmp.n_rem = 0;
    __syncthreads();
    for (int i = tid; i < t0; i += NT) {
        const int sfx = S[i];
        if (sfx >= a0) { const int at = atomicAdd(&tmp.n_rem, 1); tmp.rem[at] = i; tmp.rem_suf[at] = sfx; }
    }
    __syncthreads();
    const int nr = tmp.n_rem;
    {
        const int v = tid < nr ? tmp.rem[tid] : 0, vs = tid < nr ? tmp.rem_suf[tid] : 0;
        int rk = 0;
        for (int x = 0; x < nr; ++x) rk += tmp.rem[x] < v ? 1 : 0;
        __syncthreads();
        if (tid < nr) { tmp.rem[rk] = v; tmp.rem_suf[rk] = vs; }
    }
    __syncthreads();
    // Place of every moved suffix among the kept entries: eight lanes per suffix, binary search
    // over the old order with the taken-out entries skipped; a comparison takes eight tokens per
    // round.  Every entry between the bounds shares with the suffix at least the shorter of the
    // two prefixes it shares with the bounds (llo, lhi), so a comparison starts behind that many
    // tokens.  A suffix that was in the order before only grew, so its new place is not before
    // its old one: its search starts there.
    for (int a_base = 0; a_base < nA; a_base += NT / 8) {
        const int ai = a_base + (tid >> 3), gl = tid & 7, gsh = lane & ~7;
        const bool active = ai < nA;
        const int a = a0 + ai;
        int lo = 0, hi = active ? t0 : 0, llo = 0, lhi = 0;
        bool lo_moved = false, hi_moved = false;
        if (active && a < t0)
            for (int x = 0; x < nr; ++x) if (tmp.rem_suf[x] == a) lo = tmp.rem[x];
        for (int it = 0; it < 64 && __any_sync(0xffffffffu, lo < hi); ++it) {
            const bool busy = lo < hi;
            const int mid = (lo + hi) >> 1;
            int m2 = mid;                                       // kept entry at or behind mid, inside [mid, hi)
            if (busy) while (m2 < hi && S[m2] >= a0) ++m2;
            const bool valid = busy && m2 < hi;
            const int b = valid ? S[m2] : 0;
            int l = min(llo, lhi);
            bool less = b < a, decided = !valid;                // equal D-token strings go by position
            while (__any_sync(0xffffffffu, !decided)) {
                const int i = l + gl;
                const bool look = !decided && i < D;
                const int xb = look ? suf_tok(tx, t1, b, i) : 0, xa = look ? suf_tok(tx, t1, a, i) : 0;
                const unsigned mine = (__ballot_sync(0xffffffffu, xb != xa) >> gsh) & 0xffu;
                const int f = mine ? __ffs(mine) - 1 : 0;
                const int yb = __shfl_sync(0xffffffffu, xb, gsh + f), ya = __shfl_sync(0xffffffffu, xa, gsh + f);
                if (!decided) {
                    if (mine) { less = yb < ya; l += f; decided = true; }
                    else { l += 8; if (l >= D) { l = D; decided = true; } }
                }
            }
            if (valid) { if (less) { lo = m2 + 1; llo = l; lo_moved = true; } else { hi = mid; lhi = l; hi_moved = true; } }
            else if (busy) hi = mid;
        }
        if (active && gl == 0) {
            int before = 0;
            for (int x = 0; x < nr; ++x) before += tmp.rem[x] < lo ? 1 : 0;
            tmp.r[ai] = lo - before;
            tmp.lmin[ai] = (lo_moved && hi_moved) ? min(llo, lhi) : 0;
        }
    }
    __syncthreads();
    // order among the moved ones, and the sorted list of their places
    if (tid < nA) {
        const int a = a0 + tid, ra = tmp.r[tid];
        int o = 0, rank = 0;
        for (int bi = 0; bi < nA; ++bi) {
            const int rb = tmp.r[bi];
            // (two suffixes in the same gap share at least what each shares with both of its neighbours)
            if (rb < ra || (rb == ra && bi != tid && suf_less_from(tx, t1, D, a0 + bi, a, min(tmp.lmin[bi], tmp.lmin[tid])))) ++o;
            if (rb < ra || (rb == ra && bi < tid)) ++rank;
        }
        tmp.fin[tid] = ra + o;
        tmp.rs[rank] = ra;
    }
    __syncthreads();
    // The merged order.  A warp takes a stretch of the old order, 32 entries at a time: the index
    // of an entry among the kept ones and the moved suffixes in front of it are running counts.
    // The stretch is read from S into registers first (S is then overwritten in place); a text
    // too long for that is read from g_old instead.
    {
        constexpr int RT = 16;                                  // tiles a warp can hold in registers
        const int per = ((t0 + WARPS - 1) / WARPS + 31) & ~31;  // entries per warp
        const int i_lo = wib * per, i_hi = min(t0, i_lo + per);
        const bool in_regs = per <= 32 * RT;
        int v[RT];
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < RT; ++u) { const int i = i_lo + u * 32 + lane; v[u] = i < i_hi ? S[i] : 0x7fffffff; }
        }
        __syncthreads();
        int before = 0, ins = 0;                                // taken-out entries before the tile; moved suffixes with r < its first kept index
        for (int x = 0; x < nr; ++x) before += tmp.rem[x] < i_lo ? 1 : 0;
        while (ins < nA && tmp.rs[ins] < i_lo - before) ++ins;
        auto tile = [&](int base, int sfx) {
            const bool keep = sfx < a0;
            const unsigned km = __ballot_sync(0xffffffffu, keep);
            const int j = base - before + __popc(km & ((1u << lane) - 1u));     // index among the kept entries
            const int j_last = base - before + __popc(km) - 1;
            int add = ins;                                      // moved suffixes with r <= j come before this entry
            for (int q = ins; q < nA && tmp.rs[q] <= j_last; ++q) add += tmp.rs[q] <= j ? 1 : 0;
            if (keep) { S[j + add] = sfx; g_new[j + add] = sfx; }
            while (ins < nA && tmp.rs[ins] <= j_last) ++ins;
            before += 32 - __popc(km);
        };
        if (in_regs) {
#pragma unroll
            for (int u = 0; u < RT; ++u) if (i_lo + u * 32 < i_hi) tile(i_lo + u * 32, v[u]);
        } else {
            for (int base = i_lo; base < i_hi; base += 32) {
                const int i = base + lane;
                tile(base, i < i_hi ? g_old[i] : 0x7fffffff);
            }
        }
    }
    for (int ai = tid; ai < nA; ai += NT) {
        const int f = tmp.fin[ai];
        S[f] = a0 + ai;
        g_new[f] = a0 + ai;
    }
    __syncthreads();
}

// Range of the suffixes that start with the p tokens tx[q .. q + p) (whole warp): [lo, hi) in S.
// lo: binary search; hi: galloping from lo (ranges are mostly short), then binary search.
__device__ __forceinline__ int pat_cmp_warp(const int* tx, int t, int s, int q, int p, int lane) {
    // -1: suffix s < pattern, 0: suffix s starts with the pattern, +1: suffix s > pattern
    const int xs = lane < p ? suf_tok(tx, t, s, lane) : 0, xp = lane < p ? tx[q + lane] : 0;
    const unsigned diff = __ballot_sync(0xffffffffu, xs != xp);
    if (!diff) return 0;
    const int f = __ffs(diff) - 1;
    return __shfl_sync(0xffffffffu, xs, f) < __shfl_sync(0xffffffffu, xp, f) ? -1 : 1;
}

// First suffix in S that is not smaller than the pattern: where the pattern's range begins.
__device__ inline int pattern_lo_warp(const int* tx, int t, const int* S, int q, int p, int lane) {
    int lo = 0, hi = t;
    for (int it = 0; it < 40 && lo < hi; ++it) {
        const int mid = (lo + hi) >> 1;
        if (pat_cmp_warp(tx, t, S[mid], q, p, lane) < 0) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// First index at or behind lo whose suffix does not start with the pattern: where the range ends.
__device__ inline int pattern_hi_warp(const int* tx, int t, const int* S, int q, int p, int lo, int lane) {
    int step = 1, good = lo - 1, bad = t;                       // S[good] starts with it (or good = lo - 1), S[bad] does not (or bad = t)
    for (int it = 0; it < 40; ++it) {
        const int probe = good + step;
        if (probe >= t) break;
        if (pat_cmp_warp(tx, t, S[probe], q, p, lane) == 0) { good = probe; step <<= 1; }
        else { bad = probe; break; }
    }
    for (int it = 0; it < 40 && bad - good > 1; ++it) {
        const int mid = (good + bad) >> 1;
        if (pat_cmp_warp(tx, t, S[mid], q, p, lane) == 0) good = mid; else bad = mid;
    }
    return good + 1;
}

}  // namespace
