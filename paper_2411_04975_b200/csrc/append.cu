// Batched append kernel (sd_append): see append_core.cuh for how one token is appended.
#include "append_core.cuh"

namespace {

// Warp 0 of the grid inserts whole sequences into the global tree, one after the
// other; warp i + 1 appends item i to its request slot.
// The blocks behind those run ahead of warp 0 through the global tree: thread per token position of
// every sequence that is being inserted, walking the up to D tokens that start there, reading
// only.  The global tree is hundreds of megabytes and cold; warp 0, which has to take the tokens
// one after the other, then finds most of what it needs in L2.  Nothing is decided here.
__global__ void append_kernel(sd_store sv, int n, const int32_t* d_slot, const int64_t* d_offsets,
                              const int32_t* d_tokens, const uint8_t* d_reset, int main_blocks) {
    const int lane = threadIdx.x & 31;
    if ((int)blockIdx.x >= main_blocks) {
        const long long tid = (long long)(blockIdx.x - main_blocks) * blockDim.x + threadIdx.x;
        const long long nthreads = (long long)(gridDim.x - main_blocks) * blockDim.x;
        int seen = 0;
        for (int i = 0; i < n; ++i) {
            if (d_slot[i] != -1) continue;
            const long long b = d_offsets[i], e = d_offsets[i + 1];
            for (long long k = b + tid; k < e; k += nthreads) {
                int x = d_tokens[k];
                if (x < 0 || x >= sv.V) continue;
                int node = sv.g_root[x];
                for (int d = 1; d < sv.D && node >= 0 && k + d < e; ++d) {
                    x = d_tokens[k + d];
                    const int4 pe = sv.g_ent[node];
                    const int nc = (int)((unsigned)pe.w & RUN_COUNT_MASK);
                    int pos;
                    int4 fe;
                    node = nc > 0 ? lookup_child<8>(sv.g_ent, pe.z, nc, x, pos, fe) : -1;
                    seen += pos;
                }
            }
        }
        if (seen == 0x7fffffff) sv.g_state->status |= 0x40000000;   // keeps the loads alive; never true
        return;
    }
    const int warp = (int)((blockIdx.x * (long long)blockDim.x + threadIdx.x) >> 5);
    if (warp > n) return;
    if (warp == 0) {
        TreeRef tr{sv.g_ent, sv.g_root, (int)sv.g_cap};
        int used = sv.g_state->used, live = sv.g_state->live, status = sv.g_state->status;
        long long tokens = sv.g_state->tokens;
        bool any = false;
        for (int i = 0; i < n; ++i) {
            if (d_slot[i] != -1) continue;
            any = true;
            int act = -1, room = 0, run_cb = 0;
            unsigned run_w = 0;
            const long long b = d_offsets[i], e = d_offsets[i + 1];
            int seen = 0;
            for (long long k = b; k < e && !(status & SD_STATUS_GLOBAL_FULL); ++k) {
                if (((k - b) & 31) == 0) seen |= warm_shallow(tr, sv.V, d_tokens, b, e, k, lane);
                const int x = d_tokens[k];
                if (x < 0 || x >= sv.V) { status |= SD_STATUS_BAD_TOKEN; break; }
                if (!append_token(tr, sv.D, x, (int)(k - b), lane, act, room, run_cb, run_w, used, live)) {
                    status |= SD_STATUS_GLOBAL_FULL;
                    break;
                }
                ++tokens;
            }
            if (__any_sync(0xffffffffu, seen == 0x7fffffff)) status |= 0x40000000;   // never true
        }
        if (any && lane == 0) {
            sv.g_state->epoch += 1;                  // cached match nodes of every slot are stale now
            sv.g_state->used = used; sv.g_state->live = live; sv.g_state->status = status;
            sv.g_state->tokens = tokens;
        }
        return;
    }
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
    const unsigned ahead = 32;                                   // blocks that only warm the caches for warp 0
    append_kernel<<<blocks + ahead, warps_per_block * 32, 0, (cudaStream_t)stream>>>(*s, n, d_slot, d_offsets, d_tokens,
                                                                                     d_reset, (int)blocks);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
