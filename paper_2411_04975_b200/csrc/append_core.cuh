// Online update of the suffix trees: device functions shared by the kernels that append tokens
// (the batched append kernel, the fused decode-step kernel and the global insert kernel, which
// uses the look-up and insert primitives).
//
// Online update of the suffix trees (Section 3, "Suffix Tree Construction": the
// tokens of the ongoing request are added as they are generated, a finished
// request's output is added to the global tree).
//
// Per-request trees: one warp owns one tree for the duration of the kernel.  Appending token x at
// context length t adds one occurrence to every string that ends at x and is at
// most D tokens long: lane L extends the ACTIVE node of depth L (the node of
// the last L tokens; lane 0 extends the root) by child x, creating it or
// raising its count.  The 32 lanes work on 32 different parents at once.
//
// Placement.  A suffix that has left the known text creates one new leaf per appended token,
// each the only child of the previous one.  The first such leaf reserves room for the whole
// chain down to depth D and every later leaf goes directly behind its parent, so chains of
// only children are consecutive entries (what the wide window loads of sd_speculate exploit).
#pragma once

#include "common.cuh"

namespace {

struct TreeRef {
    int4* ent;
    int32_t* root;
    int cap;                 // entries in the pool
};

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
    const int4 ne = make_int4(x, 1, 0, 0);
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
    *word(&ent[parent], 3) = n + 1;               // dynamic run from now on (no RUN_STATIC)
    return idx;
}

// The same insert done by the whole warp for a long run (all arguments warp-uniform):
// entries move 32 at a time instead of one by one.
template <bool CG = false>
__device__ int insert_child_warp(int4* ent, int parent, int cb, int n, int pos, int x, int fresh, bool moves, int lane) {
    const int4 ne = make_int4(x, 1, 0, 0);
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
    if (lane == 0) *word(&ent[parent], 3) = n + 1;
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

// All 32 lanes call.  `act` is this lane's active node of depth lane + 1 (-1: none);
// on return it is the active node after x was appended.  `t` is the context length
// before the append.  `used` / `live` are warp-uniform pool counters.
// Returns false, changing nothing, if the pool cannot hold the new nodes.
// (run_cb, run_w) travel with `act`: the active node's child run as of now, so that the
// next token's look-up starts at the run itself instead of first reading the node.
template <int G = 8>
__device__ bool append_token(const TreeRef& tr, int D, int x, int t, int lane, int& act, int& room, int& run_cb,
                             unsigned& run_w, int& used, int& live) {
    const unsigned FULL = 0xffffffffu;
    const int parent = __shfl_up_sync(FULL, act, 1);            // node of depth `lane`
    const int parent_room = __shfl_up_sync(FULL, room, 1);      // free entries reserved behind it
    const int parent_cb = __shfl_up_sync(FULL, run_cb, 1);
    const unsigned parent_w = __shfl_up_sync(FULL, run_w, 1);
    const bool valid = lane <= min(t, D - 1);
    int found = -1, pos = 0, cb = 0, n = 0;
    unsigned w = 0;
    int4 fe = make_int4(0, 0, 0, 0);                             // the child's entry when found
    if (valid) {
        if (lane == 0) {
            found = tr.root[x];
            if (found >= 0) fe = tr.ent[found];
        } else {
            cb = parent_cb; w = parent_w;
            if (w == RUN_UNKNOWN) { const int4 pe = tr.ent[parent]; cb = pe.z; w = (unsigned)pe.w; }
            n = (int)(w & RUN_COUNT_MASK);
            found = lookup_child<G>(tr.ent, cb, n, x, pos, fe);
        }
    }
    const bool need = valid && found < 0;
    int asz = 0;                                                 // fresh entries this lane needs
    bool behind_parent = false;                                  // the new leaf goes to parent + 1
    int new_room = 0;
    if (need) {
        if (lane == 0 || n == 0) {
            // first child of a leaf (or a new depth-1 node): start or continue a chain block
            if (lane > 0 && parent_room > 0) { behind_parent = true; new_room = parent_room - 1; }
            else { asz = D - lane; new_room = asz - 1; }
        } else if ((uint32_t)n == sd_run_capacity(w)) {
            asz = (int)sd_pow2ceil((uint32_t)n + 1u);
        }
    }
    int inc = asz;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += y;
    }
    const int total = __shfl_sync(FULL, inc, 31);
    if ((long long)used + total > (long long)tr.cap) return false;
    const int fresh = behind_parent ? parent + 1 : used + inc - asz;
    const bool moves = behind_parent || asz > 0;
    used += total;

    // A lane that moves entries of its run must not do so while the next lane edits the
    // header of an entry inside that run (only possible when the last tokens repeat one
    // token): it then waits for that lane, see the rounds below.
    const int next_parent = __shfl_down_sync(FULL, parent, 1);
    const int next_need = __shfl_down_sync(FULL, need ? 1 : 0, 1);
    const bool clash = need && lane >= 1 && lane < 31 && next_need && next_parent >= cb && next_parent < cb + n;

    if (valid && found >= 0) {
        // a count changes: the copies in the run's top block (if any) are stale from now on
        if (lane > 0 && (w & RUN_HAS_TOP)) *word(&tr.ent[parent], 3) = (int)(w & ~RUN_HAS_TOP);
        *word(&tr.ent[found], 1) = fe.y + 1;
        act = found;
        run_cb = fe.z;
        run_w = (unsigned)fe.w;
        // the next lane works on this very node's run (new child, or flag dropped): what was read may be stale
        if (lane < 31 && next_parent == found) run_w = RUN_UNKNOWN;
        else if (run_w & RUN_COUNT_MASK) {
            // The next token's look-up starts in this run: ask L2 for what its first round will
            // read (the whole run if it is short, else the seven probes of an eight-way split).
            const int nn = (int)(run_w & RUN_COUNT_MASK);
            asm volatile("prefetch.global.L2 [%0];" ::"l"(tr.ent + run_cb));
            if (nn > G) {
                const int step = G == 8 ? (nn >> 3) : ((nn + 7) >> 3);
#pragma unroll
                for (int k = 0; k < 7; ++k) {
                    const int q = G == 8 ? (k + 1) * step : (k + 1) * step - 1;
                    if (q < nn) asm volatile("prefetch.global.L2 [%0];" ::"l"(tr.ent + run_cb + q));
                }
            }
        }
    } else {
        run_cb = 0;
        run_w = 0;                                               // a new leaf (or no node at all)
    }
    room = new_room;
    // Inserts run in rounds: a lane whose insert would move an entry that the next lane still has
    // to edit waits for that lane (deepest first); everybody else goes at once.  Almost always
    // there is one round; a tail of k equal tokens needs up to k.
    unsigned pend = __ballot_sync(FULL, need);
    for (int round = 0; round < 33 && pend; ++round) {
        const bool next_pending = lane < 31 && ((pend >> (lane + 1)) & 1u);
        const bool ready = need && ((pend >> lane) & 1u) && !(clash && next_pending);
        // inserts that move many entries are done by the whole warp, one after the other
        const bool big = ready && lane > 0 && (moves ? n : n - pos) > 48;
        if (ready && !big) {
            if (lane == 0) {
                tr.ent[fresh] = make_int4(x, 1, 0, 0);
                tr.root[x] = fresh;
                act = fresh;
            } else {
                act = insert_child<G>(tr.ent, parent, cb, n, pos, x, fresh, moves);
            }
        }
        __syncwarp();
        unsigned bm = __ballot_sync(FULL, big);
        while (bm) {
            const int src = __ffs(bm) - 1;
            bm &= bm - 1;
            const int idx = insert_child_warp(tr.ent, __shfl_sync(FULL, parent, src), __shfl_sync(FULL, cb, src),
                                              __shfl_sync(FULL, n, src), __shfl_sync(FULL, pos, src), x,
                                              __shfl_sync(FULL, fresh, src), __shfl_sync(FULL, moves ? 1 : 0, src) != 0,
                                              lane);
            if (lane == src) act = idx;
        }
        pend &= ~__ballot_sync(FULL, ready);
        __syncwarp();
    }
    if (!valid) { act = -1; room = 0; run_cb = 0; run_w = 0; }
    live += __popc(__ballot_sync(FULL, need));
    return true;
}

}  // namespace
