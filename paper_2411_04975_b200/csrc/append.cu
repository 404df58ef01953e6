// sd_append: the batched append kernel for the per-request trees (see append_core.cuh for how one
// token is appended) and the level-by-level insert of whole sequences into the global tree.
#include <cooperative_groups.h>

#include "append_core.cuh"

namespace cg = cooperative_groups;

namespace {

// ---------------------------------------------------------------------------------------------
// Global online insert (a finished request's output goes into the global tree), level by level.
//
// Inserting a sequence adds one occurrence to every string of at most D tokens that starts at one
// of its positions: one root-to-depth-D PATH per start position.  Taking the tokens one after the
// other makes a chain as long as the sequence.  Here up to 2,048 paths are taken at once, a
// thread per path, and all of them go down one level per round:
//   1. every path enters its current node (the parent of the node it is about to reach) into a
//      hash set in shared memory, which counts the paths per parent;
//   2. every path looks its next token up in the parent's child run.  A child that exists gets its
//      count raised by an atomic add.  A missing child is inserted at once if the path is the
//      only one at that parent: nobody else reads or writes that run during this level;
//   3. the other missing children are PENDING and are served in rounds: the waiting paths look
//      again (an earlier round may have added the very child), then per parent one path is
//      elected (a turn counter in the parent's hash-set cell) and inserts.  Runs of different
//      parents are disjoint, so the elected paths do not disturb one another;
//   4. an insert shifts or moves its run, so every path that shares its parent and whose parent's
//      run changed after it took its child looks the child's new place up.
// Only runs of ONE depth change during a level, and the entries of their parents (one level up)
// stay where they are, which is what makes the election by parent sufficient.  A node's own
// child run (first entry and size, as read with the node's entry) stays valid until the next
// level, so it travels with the path and the next look-up starts at the run itself.  There is
// no waiting on another thread anywhere, only block-wide barriers.  Placement follows the
// token-by-token append: the first leaf of a path that leaves the known text reserves room down
// to depth D and the later leaves go directly behind their parents.
//
// The block is a CLUSTER of GI_CTAS thread blocks on as many SMs (the work of a level is mostly
// instruction issue, which one SM's schedulers limit): the barriers are cluster barriers, the
// parent set is spread over the blocks' shared memories and the pool counters live in block 0's,
// all reached through distributed shared memory.  Tree entries are read through L2 (an SM's L1
// does not see what the other SMs store), and every block derives the list of sequences from
// the call's arguments for itself, so all blocks take the same branches and meet at every barrier.
constexpr int GI_CTAS = 8;
constexpr int GI_THREADS = 256;               // per block
constexpr int GI_PASS = GI_CTAS * GI_THREADS; // paths per pass
constexpr int GI_CELLS = 512;                 // cells of the parent set per block: the set is at most half full
constexpr int GI_SLOTS = GI_CTAS * GI_CELLS;
constexpr int GI_ITEMS = 256;
constexpr int GI_BIG = 48;                    // inserts that move more entries are done by a whole warp

struct GiShared {
    // the parent set, one for the odd and one for the even levels (a level clears the other one's)
    int key[2][GI_CELLS];                     // parent + 1 (level 1: token + 1), 0 = free
    int cnt[2][GI_CELLS];                     // paths at that parent
    int turn[2][GI_CELLS];                    // rounds in which a path of that parent was elected
    int item[GI_ITEMS];
    long long begin[GI_ITEMS], end[GI_ITEMS], pref[GI_ITEMS + 1];
    int n_items;
    int any[3];                               // flags of the cluster-wide "or", used in turn
    // block 0's copy only:
    unsigned long long used;
    int live, status;
};

struct GiCluster {
    cg::cluster_group cl;
    GiShared* sh;                             // this block's
    GiShared* sh0;                            // block 0's
    int phase;
    __device__ int* cell_ptr(int* base, int cell) const {       // base: a table of this block's GiShared
        return cl.map_shared_rank(base, (unsigned)cell / GI_CELLS) + (cell & (GI_CELLS - 1));
    }
    // Bit 0: a holds for any thread of the cluster, bit 1: b does.  A barrier for the whole
    // cluster.  Every block tells every block (thread r writes to block r), so the answer is read
    // from the block's own shared memory.
    __device__ int any(bool a, bool b = false) {
        const int mine = (__syncthreads_or(a) ? 1 : 0) | (__syncthreads_or(b) ? 2 : 0);
        if (threadIdx.x < GI_CTAS && mine) atomicOr(cl.map_shared_rank(&sh->any[phase], threadIdx.x), mine);
        cl.sync();
        const int r = *(volatile int*)&sh->any[phase];
        // the flag of the round before: everybody read it before arriving at the barrier above,
        // and it is written again only after the next barrier
        if (threadIdx.x == 0) sh->any[(phase + 2) % 3] = 0;
        phase = (phase + 1) % 3;
        return r;
    }
};

// Entries for new runs and chain blocks of a warp's lanes (`size` may be 0): one atomic per warp.
// Returns the lane's first entry, -1 if it asked for none or the pool cannot hold the warp's
// request (then the status bit is set as well).  All 32 lanes call.
__device__ __forceinline__ int gi_alloc_warp(GiShared* sh0, long long cap, int size, int lane) {
    const unsigned FULL = 0xffffffffu;
    int inc = size;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(FULL, inc, o);
        if (lane >= o) inc += y;
    }
    const int total = __shfl_sync(FULL, inc, 31);
    if (total == 0) return -1;
    unsigned long long at = 0;
    if (lane == 31) at = atomicAdd(&sh0->used, (unsigned long long)total);
    at = __shfl_sync(FULL, at, 31);
    if (at + (unsigned long long)total > (unsigned long long)cap) {
        if (lane == 31) atomicOr(&sh0->status, SD_STATUS_GLOBAL_FULL);
        return -1;
    }
    return size > 0 ? (int)at + inc - size : -1;
}

// Child x of `cur` is missing and this path may add it (`ins`; lanes without an insert pass
// false).  All 32 lanes call.  On return nxt is the new node and new_room the room reserved
// behind it; (seen_cb, seen_n) describe the parent's run right after the insert.  A path whose
// entries the pool cannot hold stops (rem = 0).
__device__ __forceinline__ void gi_insert(GiShared* sh0, const sd_store& sv, int d, int lane, bool ins, int x, int cur,
                                          int room, int cb, int nc, unsigned w, int pos, int& nxt, int& new_room,
                                          int& seen_cb, int& seen_n, int& rem, int& my_live) {
    const unsigned FULL = 0xffffffffu;
    int4* const ent = sv.g_ent;
    const int D = sv.D;
    bool moves = false, behind = false;
    int asz = 0;
    if (ins) {
        if (d == 1) asz = D;                                     // a new depth-1 node starts a chain block
        else if (nc == 0) {                                      // first child of a leaf: continue the chain block, or start one
            moves = true;
            if (room > 0) behind = true; else asz = D - d + 1;
        } else if ((uint32_t)nc == sd_run_capacity(w)) {         // the run is full: it moves to twice the room
            moves = true;
            asz = (int)sd_pow2ceil((uint32_t)nc + 1u);
        }
    }
    int fresh = gi_alloc_warp(sh0, sv.g_cap, asz, lane);
    bool big = false;
    if (ins) {
        if (asz > 0 && fresh < 0) rem = 0;
        else {
            ++my_live;
            if (d == 1) {
                ent[fresh] = make_int4(x, 1, 0, 0);
                sv.g_root[x] = fresh;
                nxt = fresh;
                new_room = D - 1;
            } else {
                if (behind) { fresh = cur + 1; new_room = room - 1; }
                else new_room = nc == 0 ? asz - 1 : 0;
                seen_cb = moves ? fresh : cb;
                seen_n = nc + 1;
                big = (moves ? nc : nc - pos) > GI_BIG;
                if (!big) nxt = insert_child<8, true>(ent, cur, cb, nc, pos, x, fresh, moves);
            }
        }
    }
    // inserts that move many entries: the warp does them one after the other
    unsigned bm = __ballot_sync(FULL, big);
    while (bm) {
        const int src = __ffs(bm) - 1;
        bm &= bm - 1;
        const int idx = insert_child_warp<true>(ent, __shfl_sync(FULL, cur, src), __shfl_sync(FULL, cb, src),
                                                __shfl_sync(FULL, nc, src), __shfl_sync(FULL, pos, src),
                                                __shfl_sync(FULL, x, src), __shfl_sync(FULL, fresh, src),
                                                __shfl_sync(FULL, moves ? 1 : 0, src) != 0, lane);
        if (lane == src) nxt = idx;
    }
}

__global__ void __cluster_dims__(GI_CTAS, 1, 1) __launch_bounds__(GI_THREADS, 1)
global_insert_kernel(sd_store sv, int n, const int32_t* d_slot, const int64_t* d_offsets, const int32_t* d_tokens) {
    __shared__ GiShared sh;
    const unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31;
    int4* const ent = sv.g_ent;
    const int D = sv.D;

    // (every block looks at all items: all blocks of the cluster take the same way)
    bool mine = false;
    for (int i = tid; i < n; i += GI_THREADS) mine |= d_slot[i] == -1;
    if (!__syncthreads_or(mine)) return;                         // the usual decode step: nothing for the global tree
    GiCluster G{cg::this_cluster(), &sh, nullptr, 0};
    G.sh0 = G.cl.map_shared_rank(&sh, 0);
    GiShared* const sh0 = G.sh0;
    const int path0 = (int)G.cl.block_rank() * GI_THREADS + tid; // this thread's path within a pass
    if (tid == 0) {
        sh.used = (unsigned long long)sv.g_state->used; sh.live = 0; sh.status = sv.g_state->status;
        sh.any[0] = sh.any[1] = sh.any[2] = 0;
    }
    for (int i = tid; i < 2 * GI_CELLS; i += GI_THREADS) { sh.key[0][i] = 0; sh.cnt[0][i] = 0; sh.turn[0][i] = 0; }
    G.cl.sync();
    long long tokens_done = 0;
    int my_live = 0;

    for (int base = 0; base < n; base += GI_ITEMS) {
        if (G.any((*(volatile int*)&sh0->status & SD_STATUS_GLOBAL_FULL) != 0)) break;
        // the sequences among items [base, base + GI_ITEMS), in item order
        if (tid == 0) sh.n_items = 0;
        __syncthreads();
        if (tid < 32) {
            for (int i0 = 0; i0 < GI_ITEMS; i0 += 32) {
                const int i = base + i0 + lane;
                const bool is = i < n && d_slot[i] == -1;
                const unsigned m = __ballot_sync(FULL, is);
                if (is) sh.item[sh.n_items + __popc(m & ((1u << lane) - 1u))] = i;
                __syncwarp();
                if (lane == 0) sh.n_items += __popc(m);
                __syncwarp();
            }
        }
        __syncthreads();
        const int n_items = sh.n_items;
        if (n_items == 0) continue;
        for (int j = tid; j < n_items; j += GI_THREADS) { sh.begin[j] = d_offsets[sh.item[j]]; sh.end[j] = d_offsets[sh.item[j] + 1]; }
        __syncthreads();
        // a token outside the vocabulary ends its sequence there
        for (int j = 0; j < n_items; ++j) {
            const long long b = sh.begin[j], e = d_offsets[sh.item[j] + 1];
            for (long long k = b + tid; k < e; k += GI_THREADS) {
                const int x = d_tokens[k];
                if (x < 0 || x >= sv.V) { atomicMin(&sh.end[j], k); atomicOr(&sh0->status, SD_STATUS_BAD_TOKEN); }
            }
        }
        __syncthreads();
        if (tid == 0) {
            long long acc = 0;
            for (int j = 0; j < n_items; ++j) { sh.pref[j] = acc; acc += max(sh.end[j] - sh.begin[j], 0ll); }
            sh.pref[n_items] = acc;
        }
        __syncthreads();
        const long long total = sh.pref[n_items];

        for (long long c0 = 0; c0 < total; c0 += GI_PASS) {
            // both parent sets are empty behind this barrier (the last level of a pass leaves its own behind)
            for (int i = tid; i < 2 * GI_CELLS; i += GI_THREADS) { sh.key[0][i] = 0; sh.cnt[0][i] = 0; sh.turn[0][i] = 0; }
            if (G.any((*(volatile int*)&sh0->status & SD_STATUS_GLOBAL_FULL) != 0)) break;
            // this thread's path: start position k, `rem` tokens to take (at most D)
            const long long p = c0 + path0;
            long long k = 0;
            int rem = 0;
            if (p < total) {
                int lo = 0, hi = n_items - 1;                    // last item whose prefix is <= p
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (sh.pref[mid] <= p) lo = mid; else hi = mid - 1;
                }
                k = sh.begin[lo] + (p - sh.pref[lo]);
                rem = (int)min((long long)D, sh.end[lo] - k);
            }
            // the node of the tokens taken so far, the room reserved behind it, its child run
            int cur = -1, room = 0, run_cb = 0;
            unsigned run_w = 0;
            bool more = true;                                    // a path of the cluster has a token for this level
            for (int d = 1; d <= D && more; ++d) {
                int* const t_key = sh.key[d & 1];
                int* const t_cnt = sh.cnt[d & 1];
                int* const t_turn = sh.turn[d & 1];
                const bool alive = rem >= d;
                const int x = alive ? d_tokens[k + d - 1] : 0;
                // 1. the parent set
                int cell = 0;
                if (alive) {
                    const int key = (d == 1 ? x : cur) + 1;
                    cell = (int)(((unsigned)key * 2654435761u) >> 20);          // 12 bits
                    for (int probe = 0; probe < GI_SLOTS; ++probe) {
                        const int old = atomicCAS(G.cell_ptr(t_key, cell), 0, key);
                        if (old == 0 || old == key) break;
                        cell = (cell + 1) & (GI_SLOTS - 1);
                    }
                    atomicAdd(G.cell_ptr(t_cnt, cell), 1);
                }
                G.cl.sync();
                // the other level's set: last used before the barrier that ended that level, used
                // again after the one that ends this level
                for (int i = tid; i < GI_CELLS; i += GI_THREADS) {
                    sh.key[(d & 1) ^ 1][i] = 0; sh.cnt[(d & 1) ^ 1][i] = 0; sh.turn[(d & 1) ^ 1][i] = 0;
                }
                const bool alone = alive && *(volatile int*)G.cell_ptr(t_cnt, cell) == 1;
                // 2. look the token up
                int found = -1, pos = 0;
                int cb = run_cb, nc = (int)(run_w & RUN_COUNT_MASK);
                unsigned w = run_w;
                int4 fe = make_int4(0, 0, 0, 0);
                if (alive) {
                    if (d == 1) { found = __ldcg(sv.g_root + x); if (found >= 0) fe = __ldcg(ent + found); }
                    else if (nc > 0) found = lookup_child<8, true>(ent, cb, nc, x, pos, fe);
                    if (found >= 0) {
                        atomicAdd(word(&ent[found], 1), 1);
                        // a count changes: the copies in the run's top block (if any) are stale from now on
                        if (d > 1 && (w & RUN_HAS_TOP)) atomicAnd(word(&ent[cur], 3), (int)~RUN_HAS_TOP);
                    }
                }
                int nxt = found, new_room = 0;
                int seen_cb = cb, seen_n = nc;                    // the parent's run as it was when nxt was taken
                const bool own = alive && found < 0 && alone;
                gi_insert(sh0, sv, d, lane, own, x, cur, room, cb, nc, w, pos, nxt, new_room, seen_cb, seen_n, rem, my_live);
                // A node made by a path that was alone at the parent can be reached by no other path
                // of this pass, and neither can anything below it: the rest of the path is a chain
                // of new leaves, written here in one go if the room behind the node holds it.
                if (own && rem > d && new_room >= rem - d) {
                    *word(&ent[nxt], 2) = nxt + 1;
                    *word(&ent[nxt], 3) = 1;
                    for (int j = d + 1; j <= rem; ++j)
                        ent[nxt + j - d] = j < rem ? make_int4(d_tokens[k + j - 1], 1, nxt + j - d + 1, 1)
                                                   : make_int4(d_tokens[k + j - 1], 1, 0, 0);
                    my_live += rem - d;
                    rem = 0;
                }
                // 3. the other inserts: one path per parent and round.  From the second round on every
                // waiting path first looks again: the children added in the round before are found by
                // all the paths that want them at once (text that repeats itself sends many paths
                // down the same strings), and only the children still missing are competed for.
                bool pending = alive && found < 0 && !alone;
                for (int round = 0; round <= GI_PASS; ++round) {
                    const int r = G.any(pending, rem > d);
                    more = (r & 2) != 0;
                    if (!(r & 1)) break;
                    if (round > 0) {
                        if (pending) {
                            found = -1; pos = 0;
                            if (d == 1) { found = __ldcg(sv.g_root + x); if (found >= 0) fe = __ldcg(ent + found); }
                            else {
                                const int4 pe = __ldcg(ent + cur);
                                cb = pe.z; w = (unsigned)pe.w; nc = (int)(w & RUN_COUNT_MASK);
                                if (nc > 0) found = lookup_child<8, true>(ent, cb, nc, x, pos, fe);
                            }
                            if (found >= 0) {
                                atomicAdd(word(&ent[found], 1), 1);
                                nxt = found; seen_cb = cb; seen_n = nc;
                                pending = false;
                            }
                        }
                        G.cl.sync();                             // the look-ups are over before a run moves again
                    }
                    const bool win = pending && atomicCAS(G.cell_ptr(t_turn, cell), round, round + 1) == round;
                    if (win) pending = false;
                    gi_insert(sh0, sv, d, lane, win, x, cur, room, cb, nc, w, pos, nxt, new_room, seen_cb, seen_n, rem,
                              my_live);
                }
                // 4. the child's place after all inserts of this level
                if (rem >= d && d > 1 && !alone) {
                    const int4 pe = __ldcg(ent + cur);
                    const int n2 = (int)((unsigned)pe.w & RUN_COUNT_MASK);
                    if (pe.z != seen_cb || n2 != seen_n) {
                        found = n2 > 0 ? lookup_child<8, true>(ent, pe.z, n2, x, pos, fe) : -1;
                        nxt = found;
                        new_room = 0;                            // the node left its chain block
                    }
                }
                if (rem >= d && nxt < 0) rem = 0;                // cannot happen; the path stops rather than go astray
                cur = nxt;
                room = new_room;
                run_cb = found >= 0 ? fe.z : 0;                  // a node made just now has no children
                run_w = found >= 0 ? (unsigned)fe.w : 0u;
            }
            tokens_done += min((long long)GI_PASS, total - c0);
        }
    }
    G.cl.sync();
    if (my_live) atomicAdd(&sh0->live, my_live);
    G.cl.sync();                                                 // (no block leaves while its shared memory may be in use)
    if (tid == 0 && G.cl.block_rank() == 0) {
        GlobalState* gs = sv.g_state;
        gs->epoch += 1;                              // cached match nodes of every slot are stale now
        gs->used = (int)min(sh.used, (unsigned long long)sv.g_cap);
        gs->live += sh.live;
        gs->status = sh.status;
        gs->tokens += tokens_done;
    }
}

// Warp i + 1 of the grid appends item i to its request slot (items for the global tree are
// taken by global_insert_kernel).
__global__ void append_kernel(sd_store sv, int n, const int32_t* d_slot, const int64_t* d_offsets,
                              const int32_t* d_tokens, const uint8_t* d_reset) {
    const int lane = threadIdx.x & 31;
    const int warp = (int)((blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5);
    if (warp > n || warp == 0) return;
    const int i = warp - 1;
    const int slot = d_slot[i];
    if (slot < 0 || slot >= sv.R) return;
    SlotState* ss = sv.s_state + slot;
    int32_t* text = sv.s_text + (long long)slot * sv.T;
    TreeRef tr{sv.s_ent + (long long)slot * sv.spn, sv.s_root + (long long)slot * sv.V, (int)sv.spn};
    int len = ss->len, used = ss->used, live = ss->live, status = ss->status;
    int act = ss->active[lane], room = ss->room[lane], run_cb = ss->run_cb[lane];
    unsigned run_w = ss->run_w[lane];
    if (d_reset && d_reset[i]) {
        // forget the old tree: only root-table cells of tokens that occur can be set
        for (int k = lane; k < len; k += 32) tr.root[text[k]] = -1;
        __syncwarp();
        len = 0; used = 0; live = 0; status = 0; act = -1; room = 0; run_cb = 0; run_w = 0;
        if (lane == 0) ss->gen += 1;
    }
    const long long b = d_offsets[i], e = d_offsets[i + 1];
    for (long long k = b; k < e && !(status & (SD_STATUS_POOL_FULL | SD_STATUS_BAD_TOKEN)); ++k) {
        const int x = d_tokens[k];
        if (x < 0 || x >= sv.V) { status |= SD_STATUS_BAD_TOKEN; break; }
        if (len >= sv.T || !append_token(tr, sv.D, x, len, lane, act, room, run_cb, run_w, used, live)) {
            status |= SD_STATUS_POOL_FULL;
            break;
        }
        if (lane == 0) text[len] = x;
        ++len;
    }
    ss->active[lane] = act;
    ss->room[lane] = room;
    ss->run_cb[lane] = run_cb;
    ss->run_w[lane] = run_w;
    if (lane == 0) { ss->len = len; ss->used = used; ss->live = live; ss->status = status; }
}

}  // namespace

extern "C" int sd_append(sd_store* s, int32_t n, const int32_t* d_slot, const int64_t* d_offsets,
                         const int32_t* d_tokens, const uint8_t* d_reset, void* stream) {
    if (!s || n < 0) return SD_ERR_INVALID_ARG;
    SD_CHECK_DEVICE(s);
    if (n == 0) return SD_OK;
    if (!d_slot || !d_offsets) return SD_ERR_INVALID_ARG;
    const int warps_per_block = 4;
    const unsigned blocks = (unsigned)((n + 1 + warps_per_block - 1) / warps_per_block);
    // The global tree and the request trees share nothing: the insert into the global tree runs
    // beside the appends, on the store's own stream, which starts behind everything the caller's
    // stream holds so far and which the caller's stream waits for before it goes on.
    cudaStream_t st = (cudaStream_t)stream;
    SD_CUDA_OK(cudaEventRecord(s->ev_fork, st));
    SD_CUDA_OK(cudaStreamWaitEvent(s->aux, s->ev_fork, 0));
    global_insert_kernel<<<GI_CTAS, GI_THREADS, 0, s->aux>>>(*s, n, d_slot, d_offsets, d_tokens);
    SD_CUDA_OK(cudaGetLastError());
    SD_CUDA_OK(cudaEventRecord(s->ev_join, s->aux));
    append_kernel<<<blocks, warps_per_block * 32, 0, st>>>(*s, n, d_slot, d_offsets, d_tokens, d_reset);
    SD_CUDA_OK(cudaGetLastError());
    SD_CUDA_OK(cudaStreamWaitEvent(st, s->ev_join, 0));
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
