// Online update of the global suffix tree: look-up and insert primitives of the level-by-level
// insert kernel (Section 3, "Suffix Tree Construction": a finished request's output is added to
// the global tree).
//
// Placement.  A path that has left the known text creates one new leaf per token, each the only
// child of the previous one.  The first such leaf reserves room for the whole chain down to
// depth D and every later leaf goes directly behind its parent, so chains of only children are
// consecutive entries (what the wide window loads of sd_speculate exploit).
//
// Every node an insert creates, and every run it changes, carries NODE_TOUCHED from then on
// (see common.cuh): such a node is no longer described by the suffix order of the offline build.
#pragma once

#include "common.cuh"

namespace {

__device__ __forceinline__ int* word(int4* e, int k) { return reinterpret_cast<int*>(e) + k; }

// Loads of tree entries.  CG: read through L2 only, for a kernel whose blocks run on several SMs
// and update the same tree (an SM's L1 does not see the stores and atomics of the other SMs).
template <bool CG> __device__ __forceinline__ int4 ld_ent(const int4* p) { return CG ? __ldcg(p) : *p; }
template <bool CG> __device__ __forceinline__ int ld_tok(const int4* p) { return CG ? __ldcg(&p->x) : p->x; }

// Inserts child x at sorted position `pos` into the child run of `parent`
// (cb, n children, flags in w).  `fresh` > 0: the run is full and moves to
// ent[fresh ...).  Returns the new child's entry index.
// G: entries moved (or, in the look-up, read) per round.  Eight where registers are plentiful;
// the decode-step kernel, which has to share its registers with the speculation code, uses four.
template <int G, bool CG = false>
__device__ int insert_child(int4* ent, int parent, int cb, int n, int pos, int x, int fresh, bool moves) {
    const int4 ne = make_int4(x, 1, 0, (int)NODE_TOUCHED);
    int idx;
    // entries move G at a time: the loads of a round are in flight together
    if (moves) {
        for (int k0 = 0; k0 < n; k0 += G) {
            int4 t[G];
#pragma unroll
            for (int u = 0; u < G; ++u) if (k0 + u < n) t[u] = ld_ent<CG>(ent + cb + k0 + u);
#pragma unroll
            for (int u = 0; u < G; ++u) if (k0 + u < n) ent[fresh + k0 + u + (k0 + u >= pos ? 1 : 0)] = t[u];
        }
        ent[fresh + pos] = ne;
        *word(&ent[parent], 2) = fresh;
        idx = fresh + pos;
    } else {
        for (int hi = n; hi > pos; hi -= G) {                    // from the top down
            const int lo = max(pos, hi - G);
            int4 t[G];
#pragma unroll
            for (int u = 0; u < G; ++u) if (lo + u < hi) t[u] = ld_ent<CG>(ent + cb + lo + u);
#pragma unroll
            for (int u = 0; u < G; ++u) if (lo + u < hi) ent[cb + lo + u + 1] = t[u];
        }
        ent[cb + pos] = ne;
        idx = cb + pos;
    }
    *word(&ent[parent], 3) = (int)((unsigned)(n + 1) | NODE_TOUCHED);   // dynamic run from now on (no RUN_STATIC)
    return idx;
}

// The same insert done by the whole warp for a long run (all arguments warp-uniform):
// entries move 32 at a time instead of one by one.
template <bool CG = false>
__device__ int insert_child_warp(int4* ent, int parent, int cb, int n, int pos, int x, int fresh, bool moves, int lane) {
    const int4 ne = make_int4(x, 1, 0, (int)NODE_TOUCHED);
    int idx;
    if (moves) {
        for (int i = lane; i < n; i += 32) ent[fresh + i + (i >= pos ? 1 : 0)] = ld_ent<CG>(ent + cb + i);
        idx = fresh + pos;
        if (lane == 0) { ent[idx] = ne; *word(&ent[parent], 2) = fresh; }
    } else {
        for (int hi = n; hi > pos; hi -= 32) {                   // from the top down, a chunk at a time
            const int lo = max(pos, hi - 32);
            const int i = lo + lane;
            int4 e = make_int4(0, 0, 0, 0);
            if (i < hi) e = ld_ent<CG>(ent + cb + i);
            __syncwarp();
            if (i < hi) ent[cb + i + 1] = e;
            __syncwarp();
        }
        idx = cb + pos;
        if (lane == 0) ent[idx] = ne;
    }
    if (lane == 0) *word(&ent[parent], 3) = (int)((unsigned)(n + 1) | NODE_TOUCHED);
    __syncwarp();
    return idx;
}

// Look-up of child x in the sorted run ent[cb .. cb+n): insert position in `pos`, and if the
// child exists its index is returned with its entry in `fe` (else -1).  The last round reads
// whole entries, so a run of up to G children costs one round of loads.
template <int G, bool CG = false>
__device__ int lookup_child(const int4* ent, int cb, int n, int x, int& pos, int4& fe) {
    int lo = 0, hi = n;
    while (hi - lo > 256) {                                      // very long runs: 32-way, 31 probes in flight
        const int step = (hi - lo) >> 5;
        int sel = 0;
#pragma unroll
        for (int k = 0; k < 31; ++k) sel += ld_tok<CG>(ent + cb + lo + (k + 1) * step) < x ? 1 : 0;
        const int nlo = sel == 0 ? lo : lo + sel * step + 1;
        const int nhi = sel == 31 ? hi : lo + (sel + 1) * step + 1;   // keep the pivot: it may be x itself
        lo = nlo; hi = nhi;
    }
    if (G == 8) {
        while (hi - lo > 8) {                                    // eight-way down to a window of eight
            const int step = (hi - lo) >> 3;
            int sel = 0;
#pragma unroll
            for (int k = 0; k < 7; ++k) sel += ld_tok<CG>(ent + cb + lo + (k + 1) * step) < x ? 1 : 0;
            const int nlo = sel == 0 ? lo : lo + sel * step + 1;
            const int nhi = sel == 7 ? hi : lo + (sel + 1) * step + 1;
            lo = nlo; hi = nhi;
        }
    } else {
        // eight parts of `step` entries, probed at their last entries: the window becomes the
        // first part that does not lie wholly below x (32 entries or fewer leave at most four)
        while (hi - lo > G) {
            const int step = (hi - lo + 7) >> 3;
            int sel = 0;
#pragma unroll
            for (int k = 0; k < 7; ++k) {
                const int q = lo + (k + 1) * step - 1;
                sel += (q < hi && ld_tok<CG>(ent + cb + q) < x) ? 1 : 0;
            }
            lo += sel * step;
            hi = min(hi, lo + step);
        }
    }
    int4 e[G];
#pragma unroll
    for (int k = 0; k < G; ++k) e[k] = lo + k < hi ? ld_ent<CG>(ent + cb + lo + k) : make_int4(0x7fffffff, 0, 0, 0);
    int below = 0;
#pragma unroll
    for (int k = 0; k < G; ++k) below += e[k].x < x ? 1 : 0;
    pos = lo + below;
    int found = -1;
#pragma unroll
    for (int k = 0; k < G; ++k) if (k == below && lo + k < hi && e[k].x == x) { fe = e[k]; found = cb + lo + k; }
    return found;
}

}  // namespace
