// GenerateCandidateTree (Algorithm 1) for a whole batch.
//
// Kernel 1, one warp per (request, tree, p) job: MatchPattern, then
// ExpandSpeculationTree with a warp-wide sorted frontier, then SCORE (Eq. 4).
// Kernel 2, one warp per request: pick the first job with the strictly largest
// score and write the verifier's arrays (tokens, parents, positions, mask).
//
// fp64 rules: C = count / sibling-sum (Eq. 1), D = D(parent) * C (Eq. 2), SCORE
// adds D in insertion order; __ddiv_rn / __dmul_rn / __dadd_rn keep every
// operation a separately rounded IEEE binary64 operation (no FMA contraction).
#include <mutex>

#include "common.cuh"

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
__device__ __forceinline__ bool better(double da, int ta, int pa, double db, int tb, int pb) {
    if (da != db) return da > db;
    if (ta != tb) return ta < tb;
    return pa < pb;
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
__device__ void frontier_insert(Frontier& F, int fh, int& fs, int K, double d, int tok, int par, int cb, unsigned nc,
                                int lane) {
    const int i0 = lane, i1 = lane + 32;
    const int s0 = (fh + i0) & (SD_MAX_SPEC - 1), s1 = (fh + i1) & (SD_MAX_SPEC - 1);
    const bool b0 = i0 < fs && better(F.d[s0], F.tok[s0], F.par[s0], d, tok, par);
    const bool b1 = i1 < fs && better(F.d[s1], F.tok[s1], F.par[s1], d, tok, par);
    const int pos = __popc(__ballot_sync(FULL, b0)) + __popc(__ballot_sync(FULL, b1));
    if (pos >= K) return;
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

__global__ void select_emit_kernel(sd_store sv, int n, const int32_t* __restrict__ d_slot, int Pe, int32_t* d_n_draft,
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
    if (ok && best_o >= 0) {
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

}  // namespace

extern "C" int sd_speculate(sd_store* s, int32_t n, const int32_t* d_slot, const sd_spec_params* prm,
                            const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents,
                            int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
                            double* d_score, int32_t* d_status, void* stream) {
    if (!s || !prm || n < 0 || n > s->R) return SD_ERR_INVALID_ARG;
    if (prm->P < 1 || prm->max_spec < 0 || prm->max_spec > s->M || !(prm->alpha >= 0.0)) return SD_ERR_INVALID_ARG;
    if ((prm->flags & SD_FLAG_GLOBAL_ONLY) && (prm->flags & SD_FLAG_REQUEST_ONLY)) return SD_ERR_INVALID_ARG;
    if (n == 0) return SD_OK;
    if (!d_slot || !d_n_draft || !d_tokens || !d_parents || !d_positions || !d_mask || !d_chosen_tree || !d_chosen_p ||
        !d_score)
        return SD_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const int Pe = prm->P < s->D ? prm->P : s->D;               // longer patterns never match
    const long long jobs = (long long)n * 2 * Pe;
    match_expand_kernel<<<(unsigned)((jobs + SPEC_WARPS - 1) / SPEC_WARPS), SPEC_WARPS * 32, 0, st>>>(
        *s, n, d_slot, Pe, prm->alpha, prm->max_spec, prm->flags, d_budget_cap);
    select_emit_kernel<<<(unsigned)((n + 3) / 4), 128, 0, st>>>(*s, n, d_slot, Pe, d_n_draft, d_tokens, d_parents,
                                                                d_positions, d_mask, d_chosen_tree, d_chosen_p, d_score,
                                                                d_status);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
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
    if (prm->P < 1 || prm->max_spec < 0 || prm->max_spec > s->M || !(prm->alpha >= 0.0)) return SD_ERR_INVALID_ARG;
    if ((prm->flags & SD_FLAG_GLOBAL_ONLY) && (prm->flags & SD_FLAG_REQUEST_ONLY)) return SD_ERR_INVALID_ARG;
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
    select_emit_kernel<<<(unsigned)((n + 3) / 4), 128, 0, st>>>(view, n, d_slot, Pe, d_n_draft, d_tokens, d_parents,
                                                                d_positions, d_mask, d_chosen_tree, d_chosen_p, d_score,
                                                                d_status);
    SD_CUDA_OK(cudaGetLastError());
    return SD_OK;
}
