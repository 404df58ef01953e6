// Batched append kernel (sd_append): see append_core.cuh for how one token is appended.
#include "append_core.cuh"

namespace {

// ---------------------------------------------------------------------------------------------
// Global online insert (a finished request's output goes into the global tree), level by level.
//
// Inserting a sequence adds one occurrence to every string of at most D tokens that starts at one
// of its positions: one root-to-depth-D PATH per start position.  Taking the tokens one after the
// other makes a chain as long as the sequence.  Here one block takes up to 1,024 paths at once, a
// thread per path, and all of them go down one level per round:
//   A. every path looks its next token up in the child run of its current node; a child that
//      exists gets its count raised by an atomic add, the others are PENDING;
//   B. pending paths are served in rounds: per parent node one path is elected (a table of locks
//      in shared memory, indexed by a hash of the parent), looks again (an earlier round may
//      have added the very child) and inserts.  Runs of different parents are disjoint, so the
//      elected paths do not disturb one another; paths of the same parent go one per round;
//   C. an insert shifts or moves its run, so every path whose parent's run changed after it
//      found its child looks the child's new place up.
// Only runs of ONE depth change during a level, and the entries of their parents (one level up)
// stay where they are, which is what makes the election by parent sufficient.  There is no
// waiting on another thread anywhere, only block-wide barriers.  Placement follows the
// token-by-token append: the first leaf of a path that leaves the known text reserves room down
// to depth D and the later leaves go directly behind their parents.
constexpr int GI_THREADS = 1024;
constexpr int GI_LOCKS = 4096;
constexpr int GI_ITEMS = 256;
constexpr int GI_BIG = 48;                    // inserts that move more entries are done by a whole warp

struct GiShared {
    int lock[GI_LOCKS];
    int item[GI_ITEMS];
    long long begin[GI_ITEMS], end[GI_ITEMS], pref[GI_ITEMS + 1];
    unsigned long long used;
    int n_items, live, status;
};

__device__ __forceinline__ unsigned gi_hash(int key) { return ((unsigned)key * 2654435761u) >> 20; }   // 12 bits

// Entries for a new run or chain block; -1 (and the status bit) when the pool cannot hold them.
__device__ __forceinline__ int gi_alloc(GiShared& sh, long long cap, int size) {
    const unsigned long long at = atomicAdd(&sh.used, (unsigned long long)size);
    if (at + (unsigned long long)size > (unsigned long long)cap) { atomicOr(&sh.status, SD_STATUS_GLOBAL_FULL); return -1; }
    return (int)at;
}

__global__ void __launch_bounds__(GI_THREADS, 1)
global_insert_kernel(sd_store sv, int n, const int32_t* d_slot, const int64_t* d_offsets, const int32_t* d_tokens) {
    __shared__ GiShared sh;
    const unsigned FULL = 0xffffffffu;
    const int tid = threadIdx.x, lane = tid & 31;
    int4* const ent = sv.g_ent;
    int32_t* const root = sv.g_root;
    const int D = sv.D;

    bool mine = false;
    for (int i = tid; i < n; i += GI_THREADS) mine |= d_slot[i] == -1;
    if (!__syncthreads_or(mine)) return;                         // the usual decode step: nothing for the global tree
    if (tid == 0) { sh.used = (unsigned long long)sv.g_state->used; sh.live = 0; sh.status = sv.g_state->status; }
    __syncthreads();
    long long tokens_done = 0;

    for (int base = 0; base < n; base += GI_ITEMS) {
        if (__syncthreads_or(sh.status & SD_STATUS_GLOBAL_FULL)) break;
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
                if (x < 0 || x >= sv.V) { atomicMin(&sh.end[j], k); atomicOr(&sh.status, SD_STATUS_BAD_TOKEN); }
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

        for (long long c0 = 0; c0 < total; c0 += GI_THREADS) {
            if (__syncthreads_or(sh.status & SD_STATUS_GLOBAL_FULL)) break;
            // this thread's path: start position k, `rem` tokens to take (at most D)
            const long long p = c0 + tid;
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
            int cur = -1, room = 0;                              // node of the tokens taken so far; room reserved behind it
            for (int d = 1; d <= D; ++d) {
                if (!__syncthreads_or(rem >= d)) break;
                const bool alive = rem >= d;
                const int x = alive ? d_tokens[k + d - 1] : 0;
                int found = -1, pos = 0, cb = 0, nc = 0;
                unsigned w = 0;
                int4 fe = make_int4(0, 0, 0, 0);
                // A: look the token up
                if (alive) {
                    if (d == 1) found = root[x];
                    else {
                        const int4 pe = ent[cur];
                        cb = pe.z; w = (unsigned)pe.w; nc = (int)(w & RUN_COUNT_MASK);
                        if (nc > 0) found = lookup_child<8>(ent, cb, nc, x, pos, fe);
                    }
                    if (found >= 0) {
                        atomicAdd(word(&ent[found], 1), 1);
                        // a count changes: the copies in the run's top block (if any) are stale from now on
                        if (d > 1 && (w & RUN_HAS_TOP)) atomicAnd(word(&ent[cur], 3), (int)~RUN_HAS_TOP);
                    }
                }
                bool pending = alive && found < 0;
                int nxt = found, new_room = 0;
                int seen_cb = cb, seen_n = nc;                    // the parent's run as it was when nxt was taken
                // B: inserts, one path per parent and round
                for (int round = 0; round <= GI_THREADS; ++round) {
                    if (!__syncthreads_or(pending)) break;
                    for (int i = tid; i < GI_LOCKS; i += GI_THREADS) sh.lock[i] = 0;
                    __syncthreads();
                    const bool win = pending && atomicCAS(&sh.lock[gi_hash(d == 1 ? x : cur)], 0, 1) == 0;
                    bool big = false;
                    int fresh = 0;
                    bool moves = false;
                    if (win) {
                        pending = false;
                        if (round > 0) {                         // an earlier round may have changed the run
                            found = -1; pos = 0;
                            if (d == 1) found = root[x];
                            else {
                                const int4 pe = ent[cur];
                                cb = pe.z; w = (unsigned)pe.w; nc = (int)(w & RUN_COUNT_MASK);
                                if (nc > 0) found = lookup_child<8>(ent, cb, nc, x, pos, fe);
                            }
                        }
                        if (found >= 0) {                        // added meanwhile by a path with the same string
                            atomicAdd(word(&ent[found], 1), 1);
                            nxt = found; seen_cb = cb; seen_n = nc;
                        } else if (d == 1) {
                            fresh = gi_alloc(sh, sv.g_cap, D);
                            if (fresh >= 0) {
                                ent[fresh] = make_int4(x, 1, 0, 0);
                                root[x] = fresh;
                                nxt = fresh; new_room = D - 1;
                                atomicAdd(&sh.live, 1);
                            } else rem = 0;
                        } else {
                            bool ok = true;
                            if (nc == 0) {
                                // first child of a leaf: continue the chain block, or start one
                                moves = true;
                                if (room > 0) { fresh = cur + 1; new_room = room - 1; }
                                else { const int asz = D - d + 1; fresh = gi_alloc(sh, sv.g_cap, asz); new_room = asz - 1; ok = fresh >= 0; }
                            } else if ((uint32_t)nc == sd_run_capacity(w)) {
                                moves = true;
                                fresh = gi_alloc(sh, sv.g_cap, (int)sd_pow2ceil((uint32_t)nc + 1u));
                                ok = fresh >= 0;
                            }
                            if (!ok) { rem = 0; new_room = 0; }
                            else {
                                atomicAdd(&sh.live, 1);
                                seen_cb = moves ? fresh : cb; seen_n = nc + 1;
                                big = (moves ? nc : nc - pos) > GI_BIG;
                                if (!big) nxt = insert_child<8>(ent, cur, cb, nc, pos, x, fresh, moves);
                            }
                        }
                    }
                    // inserts that move many entries: the warp does them one after the other
                    unsigned bm = __ballot_sync(FULL, big);
                    while (bm) {
                        const int src = __ffs(bm) - 1;
                        bm &= bm - 1;
                        const int idx = insert_child_warp(ent, __shfl_sync(FULL, cur, src), __shfl_sync(FULL, cb, src),
                                                          __shfl_sync(FULL, nc, src), __shfl_sync(FULL, pos, src),
                                                          __shfl_sync(FULL, x, src), __shfl_sync(FULL, fresh, src),
                                                          __shfl_sync(FULL, moves ? 1 : 0, src) != 0, lane);
                        if (lane == src) nxt = idx;
                    }
                }
                // C: the child's place after all inserts of this level
                if (rem >= d && d > 1) {
                    const int4 pe = ent[cur];
                    const int n2 = (int)((unsigned)pe.w & RUN_COUNT_MASK);
                    if (pe.z != seen_cb || n2 != seen_n) {
                        nxt = n2 > 0 ? lookup_child<8>(ent, pe.z, n2, x, pos, fe) : -1;
                        new_room = 0;                            // the node left its chain block
                    }
                }
                if (rem >= d && nxt < 0) rem = 0;                // cannot happen; the path stops rather than go astray
                cur = nxt;
                room = new_room;
            }
            tokens_done += min((long long)GI_THREADS, total - c0);
        }
    }
    __syncthreads();
    if (tid == 0) {
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
    if (n == 0) return SD_OK;
    if (!d_slot || !d_offsets) return SD_ERR_INVALID_ARG;
    const int warps_per_block = 4;
    const unsigned blocks = (unsigned)((n + 1 + warps_per_block - 1) / warps_per_block);
    global_insert_kernel<<<1, GI_THREADS, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_offsets, d_tokens);
    SD_CUDA_OK(cudaGetLastError());
    append_kernel<<<blocks, warps_per_block * 32, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_offsets, d_tokens, d_reset);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
