/*
 * suffixspec: batched SuffixDecoding draft generation on one NVIDIA B200.
 *
 * C ABI.  Every pointer named d_* is DEVICE memory owned by the caller; every
 * other pointer is HOST memory.  For the per-step inputs and outputs "device
 * memory" means any address the GPU can use: page-locked host memory
 * (cudaHostAlloc / cudaHostRegister, unified addressing) is accepted as it is,
 * and the kernels then read the few KB of inputs and write the drafts across
 * the bus themselves, which saves the copies before and after a step.  A store owns all of its device memory from
 * sd_build() until sd_free().  Calls are asynchronous on `stream` (a
 * cudaStream_t passed as void*, NULL = default stream) unless stated; the
 * per-step calls (sd_append, sd_speculate) never allocate device memory.
 *
 * Return value: SD_OK (0) or a negative SD_ERR_* code.  Nothing aborts, throws
 * or traps.  Conditions that depend on device data (a request whose slot pool
 * ran full, an empty slot) are reported per request in d_status and leave the
 * store consistent.  A store belongs to the CUDA device that was current in
 * sd_build(); every call checks that this device is current (else
 * SD_ERR_INVALID_ARG).
 *
 * Limits: depth_cap <= 32, max_spec_cap <= 64, P <= depth_cap is not required
 * (pattern lengths above depth_cap or above the context length never match).
 */
#ifndef SUFFIXSPEC_H
#define SUFFIXSPEC_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sd_store sd_store;

enum {
    SD_OK = 0,
    SD_ERR_INVALID_ARG = -1,
    SD_ERR_CUDA = -2,
    SD_ERR_NOMEM = -3,
    SD_ERR_CAPACITY = -4
};

/* per-request status bits (d_status of sd_speculate, sd_slot_info) */
enum {
    SD_STATUS_OK = 0,
    SD_STATUS_BAD_SLOT = 1,       /* slot index out of range                         */
    SD_STATUS_POOL_FULL = 2,      /* the slot's node pool or text buffer ran full;    */
                                  /* its tree stopped growing at the last good token  */
    SD_STATUS_GLOBAL_FULL = 4,    /* the global node pool ran full during an insert   */
    SD_STATUS_BAD_TOKEN = 8       /* a token outside [0, V) was met; the tree stopped */
                                  /* growing at the last good token                   */
};

/* sd_spec_params.flags */
enum {
    SD_FLAG_GLOBAL_ONLY = 1,      /* speculate from the global tree only              */
    SD_FLAG_REQUEST_ONLY = 2,     /* speculate from the per-request tree only         */
    SD_FLAG_LINEAR = 4            /* chain-only expansion ("Suffix (linear)")         */
};

typedef struct {
    int32_t vocab;                /* V: token ids are in [0, V)                       */
    int32_t depth_cap;            /* D: paths longer than D tokens are not stored     */
    int32_t max_requests;         /* number of request slots                          */
    int32_t max_req_tokens;       /* max prompt + generated tokens per slot           */
    int32_t max_spec_cap;         /* M: row stride of the per-draft outputs, <= 64    */
    int64_t global_extra_nodes;   /* node head-room for online inserts into the       */
                                  /* global tree; < 0: library default                */
    int64_t slot_pool_nodes;      /* node pool per slot; <= 0: library default        */
                                  /* (2 * max_req_tokens * depth_cap)                 */
} sd_build_params;

typedef struct {
    int32_t P;                    /* max pattern length                               */
    double alpha;                 /* max speculation factor: MAX_SPEC(p) = alpha * p  */
    int32_t max_spec;             /* cap on MAX_SPEC(p), <= max_spec_cap              */
    uint32_t flags;               /* SD_FLAG_*                                        */
    double tau;                   /* score threshold of Section 3.2 ("Hybrid Suffix   */
                                  /* Speculative Decoding"): a request gets a draft   */
                                  /* only if SCORE > tau (strict); otherwise n_draft  */
                                  /* = 0, chosen_tree = -1, score = 0 and the caller  */
                                  /* falls back to its other drafter.  0: no gate     */
                                  /* beyond Algorithm 1's SCORE > 0.  Must be >= 0.   */
} sd_spec_params;

typedef struct {
    int64_t global_nodes;         /* live nodes of the global tree                    */
    int64_t global_pool_used;     /* node entries handed out (live + abandoned)       */
    int64_t global_pool_cap;
    int64_t global_tokens;        /* tokens inserted so far                           */
    int64_t slot_pool_nodes;      /* node entries per slot                            */
    int64_t device_bytes;         /* device memory owned by the store                 */
    int32_t global_status;        /* SD_STATUS_GLOBAL_FULL or 0                       */
} sd_stats_t;

/*
 * sd_build: create a store and build the GLOBAL suffix tree over a corpus of
 * previous outputs in one offline step (Section 3, "Suffix Tree Construction").
 * One node per token; the root-to-node path is a token string of at most
 * depth_cap tokens that occurs in some sequence, and the node's count is its
 * number of occurrences (COUNT as used by Eq. 1).  Strings do not cross
 * sequence boundaries.  The tree is built on the GPU by a depth-capped suffix
 * sort followed by adjacent-suffix LCPs.
 *   d_corpus       int32[seq_offsets[n_seqs]]  tokens of all sequences, back to back
 *   d_seq_offsets  int64[n_seqs + 1]           start of each sequence, ascending, [0] = 0
 * n_seqs may be 0 (empty global tree; both pointers may then be NULL).
 * Also allocates max_requests empty per-request trees.  Synchronises the stream.
 * On success *out is the new store; on failure *out is NULL and nothing leaks.
 * Errors: INVALID_ARG (NULL, limits, a corpus token outside [0, V), offsets not
 * ascending), NOMEM (cudaMalloc failed), CUDA.
 */
int sd_build(const sd_build_params* params, const int32_t* d_corpus, const int64_t* d_seq_offsets,
             int32_t n_seqs, void* stream, sd_store** out);

/*
 * sd_append: online update of the trees (Section 3, "Suffix Tree Construction":
 * tokens of the ongoing request are added as they are generated; a finished
 * request's output is added to the global tree).
 * For item i in [0, n):
 *   d_slot[i] >= 0 : append tokens d_tokens[d_offsets[i] .. d_offsets[i+1]) to the
 *                    per-request tree (and stored context) of that slot; if
 *                    d_reset[i] != 0 the slot is emptied first (new request, the
 *                    tokens are its prompt).  A slot may appear at most once per call.
 *   d_slot[i] == -1: insert the tokens as one whole sequence into the GLOBAL tree.
 * After the call each tree equals the tree built from scratch over its text.
 *   d_slot int32[n], d_offsets int64[n+1], d_tokens int32[d_offsets[n]],
 *   d_reset uint8[n] or NULL (no resets).
 * A slot whose pool or text buffer would overflow keeps its state from before
 * the offending token and gets SD_STATUS_POOL_FULL (see sd_slot_info).
 * Global tree: a sequence is inserted up to its first token outside [0, V)
 * (SD_STATUS_BAD_TOKEN in sd_stats' global_status, the other sequences of the
 * call are not affected).  When the global pool cannot hold the new nodes
 * SD_STATUS_GLOBAL_FULL is set: strings whose nodes found no room are missing
 * or counted short, the tree stays consistent and usable, and later calls
 * insert nothing more into it.  n == 0 is a no-op.
 * Stream order: for the caller everything is ordered on `stream`.  Inside the
 * call the insert into the global tree runs on a stream the store owns, which
 * starts behind the work `stream` holds at the call and which `stream` waits
 * for before it goes on (the two kinds of tree share nothing, so the insert
 * and the appends to the request trees run side by side).
 * Errors: INVALID_ARG, CUDA (launch failure).
 */
int sd_append(sd_store* store, int32_t n, const int32_t* d_slot, const int64_t* d_offsets,
              const int32_t* d_tokens, const uint8_t* d_reset, void* stream);

/*
 * sd_build_requests: start n new requests at once: their per-request trees are built from the
 * prompts by the sort-based pipeline of sd_build instead of token by token (Section 3, "Suffix
 * Tree Construction": the per-request tree is constructed when the request is received).  The
 * result is the same as sd_append with d_reset = 1 for every item, only faster for long prompts.
 *   h_slot     int32[n]    HOST: slot of each request (each slot at most once, 0 <= slot < max_requests)
 *   h_offsets  int64[n+1]  HOST: prompt i is d_tokens[h_offsets[i] .. h_offsets[i+1]), h_offsets[0] = 0
 *   d_tokens   int32[h_offsets[n]]  DEVICE
 * A prompt that does not fit the slot's node pool or text buffer leaves the slot empty with
 * SD_STATUS_POOL_FULL.  Unlike the per-step calls this one may allocate device memory: its
 * temporaries (about 100 bytes per prompt token of the largest batch so far) are kept by the
 * store and reused.  The host arrays have been read when the call returns (it synchronises the
 * stream once, after the tokens have been checked); the trees themselves are built
 * asynchronously on `stream` like any per-step call's work when the prompts hold at most 65,536
 * tokens in total (a few new requests in the middle of a decode loop), and with further
 * synchronisations above that.  The workspace is shared by all calls on a store: order calls
 * made on different streams.
 * Errors: INVALID_ARG (bad slot, slot twice, offsets not ascending, token outside [0, V): nothing
 * is changed), CAPACITY (n * vocab or the token total does not fit 31 bits), NOMEM, CUDA.
 */
int sd_build_requests(sd_store* store, int32_t n, const int32_t* h_slot, const int64_t* h_offsets,
                      const int32_t* d_tokens, void* stream);

/*
 * sd_speculate: GenerateCandidateTree of Algorithm 1 for n requests at once.
 * For each request the context x_{1:t} is the slot's stored text.  For the
 * global tree, then the per-request tree, and p = 1..P: MatchPattern walks the
 * last p tokens; ExpandSpeculationTree grows the sub-tree greedily by the
 * largest D(N) (Eq. 1, Eq. 2) up to min(floor(alpha * p), max_spec) draft nodes
 * (Eq. 3; the match node itself is not a draft); SCORE (Eq. 4) is the sum of
 * D over the draft nodes in the order added; the first tree with the strictly
 * largest score wins.  Candidate ties: larger D, then smaller token id, then
 * smaller index of the parent inside the speculation tree.  All scores are
 * IEEE binary64: divide, multiply root-to-leaf, add in insertion order, no FMA.
 * Section 3.2: the chosen tree is handed out only if its SCORE > params->tau.
 * Outputs, row stride M = max_spec_cap, draft nodes in insertion order:
 *   d_n_draft     int32[n]        number of draft nodes (0: no speculation)
 *   d_tokens      int32[n][M]     token of each draft node, -1 beyond n_draft
 *   d_parents     int32[n][M]     index of the parent draft node, -1 = child of the
 *                                 match node (also -1 beyond n_draft)
 *   d_positions   int32[n][M]     0-based sequence position t + depth - 1, -1 beyond
 *   d_mask        uint32[n][M][(M+31)/32]  bit j of row i set iff j == i or j is an
 *                                 ancestor of i (tree-attention mask), 0 beyond
 *   d_chosen_tree int32[n]        0 global, 1 per-request, -1 none
 *   d_chosen_p    int32[n]        pattern length of the chosen tree, 0 if none
 *   d_score       double[n]       SCORE of the chosen tree, 0.0 if none
 *   d_status      int32[n]        SD_STATUS_* of the request's slot
 *   d_budget_cap  int32[n] or NULL: per-request cap on the draft size (< 0: none)
 * The slots of a call must be distinct; a slot that appears twice gets
 * SD_STATUS_BAD_SLOT and no draft for its later appearances.
 * Errors: INVALID_ARG (n > max_requests, max_spec > M, P < 1, tau < 0 or NaN ...), CUDA.
 */
int sd_speculate(sd_store* store, int32_t n, const int32_t* d_slot, const sd_spec_params* params,
                 const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens, int32_t* d_parents,
                 int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
                 double* d_score, int32_t* d_status, void* stream);

/*
 * sd_step: one decode step in one launch: for every request i first append the tokens
 * d_new_tokens[d_offsets[i] .. d_offsets[i+1]) (accepted drafts + bonus token of the previous
 * step) to its per-request tree and context, then speculate, exactly as sd_append followed by
 * sd_speculate on the same slots would (Section 3: tokens are added to the per-request tree as
 * they are generated; Algorithm 1 then runs on the extended context).  The appends of requests
 * with many new tokens overlap with the speculation of the others.
 *   d_slot int32[n]: distinct slots >= 0 (no global inserts, no resets: use sd_append for those);
 *   d_offsets int64[n+1], d_new_tokens int32[d_offsets[n]]; all other arguments as sd_speculate.
 * A request whose append stops early (pool full, bad token) gets no draft and the status bits.
 */
int sd_step(sd_store* store, int32_t n, const int32_t* d_slot, const int64_t* d_offsets, const int32_t* d_new_tokens,
            const sd_spec_params* params, const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens,
            int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree, int32_t* d_chosen_p,
            double* d_score, int32_t* d_status, void* stream);

/*
 * sd_speculate_noalloc: sd_speculate for callers that must not allocate.
 * (The paper has no counterpart; this is a deployment convenience.)
 *
 * Some hosts of this library run where device allocation is off limits: a
 * serving loop that has handed all free device memory to its own pool, a
 * plug-in that is only given buffers and a stream, or a real-time thread that
 * may not take the allocator's locks.  sd_speculate needs no global scratch
 * (its one kernel keeps everything in shared memory); this variant runs the
 * library's two-kernel form of the same computation, one warp per (request,
 * tree, pattern length), whose per-job records go through global memory, and
 * keeps those records in a fixed array inside the library image instead of in
 * memory from cudaMalloc.  It calls no allocating routine at all.  Unlike
 * sd_speculate it neither uses nor refreshes the slots' cached global match
 * nodes.
 *
 * Same arguments, outputs and results as sd_speculate.  Differences:
 *  - Size limit: n * 2 * depth_cap must not exceed SD_NOALLOC_MAX_JOBS (e.g. 64
 *    requests at depth_cap 32); a larger batch returns SD_ERR_CAPACITY
 *    ("capacity exceeded") and launches nothing.  Split the batch instead.
 *  - The array (about 2.1 MB) is held on every GPU that loads the library,
 *    until the process exits.
 *  - The first call on each device looks up the array's device address (a
 *    short, synchronous runtime query; that device must be current).  Make
 *    that first call before starting any stream capture.
 *  - All calls on a device share the one array.  Its contents carry over from
 *    call to call but are never read before being rewritten, so no clearing is
 *    needed; two calls whose kernels overlap on the GPU (different streams,
 *    different stores) would overwrite each other's records, so keep calls on
 *    one device ordered.
 */
#define SD_NOALLOC_MAX_JOBS 4096
int sd_speculate_noalloc(sd_store* store, int32_t n, const int32_t* d_slot, const sd_spec_params* params,
                         const int32_t* d_budget_cap, int32_t* d_n_draft, int32_t* d_tokens,
                         int32_t* d_parents, int32_t* d_positions, uint32_t* d_mask, int32_t* d_chosen_tree,
                         int32_t* d_chosen_p, double* d_score, int32_t* d_status, void* stream);

/*
 * sd_query_counts: COUNT of arbitrary token paths (the quantity Eq. 1 divides),
 * for checking a store against an independent implementation.
 *   d_tree int32[n]: -1 global tree, else slot; path i is
 *   d_paths[d_offsets[i] .. d_offsets[i+1]); d_counts int32[n] receives the count,
 *   0 when the path is not in the tree (or is longer than depth_cap).
 */
int sd_query_counts(sd_store* store, int32_t n, const int32_t* d_tree, const int64_t* d_offsets,
                    const int32_t* d_paths, int32_t* d_counts, void* stream);

/*
 * sd_enumerate: every node of a tree as a record (parent record, token, COUNT, depth), for
 * comparing a whole tree with an independent implementation (the trees of Section 3.1 are
 * defined by exactly these: which token paths exist and how often each occurred).
 *   tree: -1 global tree, else a slot.  d_parent, d_token, d_count, d_depth: DEVICE int32[max_nodes],
 *   caller-owned.  Record i describes one node: d_parent[i] is the record of its parent (-1 for
 *   a node of depth 1) and always precedes i; d_depth[i] is 1-based.  The order of the records
 *   is otherwise unspecified and may change from call to call.  h_n: HOST, receives the number of
 *   nodes of the tree.  If that exceeds max_nodes the call returns SD_ERR_CAPACITY, *h_n still
 *   holds the number needed and the records are incomplete.
 * An offline analysis call: allocates temporary device memory (16 bytes per record of room)
 * and synchronises the stream once per level.
 */
int sd_enumerate(sd_store* store, int32_t tree, int64_t max_nodes, int32_t* d_parent, int32_t* d_token,
                 int32_t* d_count, int32_t* d_depth, int64_t* h_n, void* stream);

/*
 * sd_slot_info: per-slot context length, live node count and status.
 *   d_slot int32[n]; outputs int32[n] each, any may be NULL.
 */
int sd_slot_info(sd_store* store, int32_t n, const int32_t* d_slot, int32_t* d_len, int32_t* d_nodes,
                 int32_t* d_status, void* stream);

/*
 * sd_entropy: empirical entropy of a tree in bits (Appendix "Predicting SuffixDecoding
 * Effectiveness"): for every node that has children, the entropy of the children's count
 * distribution; the result is the average over those nodes (the root included) weighted by the
 * sum of the children's counts.  A low value says the next token is predictable from its
 * prefix, i.e. that suffix-tree speculation will work well on this kind of text.
 *   tree: -1 global tree, else a slot.  h_entropy: HOST double.  An empty tree gives 0.
 * An offline analysis call: allocates temporary device memory and synchronises the stream.
 * Sums are accumulated with atomics, so the last bits vary from call to call.
 */
int sd_entropy(sd_store* store, int32_t tree, double* h_entropy, void* stream);

/* sd_stats: store-wide figures into HOST memory.  Synchronises the stream. */
int sd_stats(sd_store* store, sd_stats_t* out, void* stream);

/* sd_free: release a store (NULL is a no-op).  Synchronises the device. */
void sd_free(sd_store* store);

/* sd_strerror: static description of an SD_* return code. */
const char* sd_strerror(int code);

/*
 * sd_debug_fail_alloc: test hook for the out-of-memory paths.  The k-th device allocation the
 * library makes from now on fails as if the device were out of memory (k = 1: the next one);
 * k = 0 switches the hook off.  sd_build must then return SD_ERR_NOMEM and leak nothing.
 */
void sd_debug_fail_alloc(int64_t k);

#ifdef __cplusplus
}
#endif
#endif /* SUFFIXSPEC_H */
