// Shared declarations of the suffixspec CUDA library (sm_100a).
//
// Node storage.  A tree node is a 16-byte ENTRY that lives inside its parent's
// child run:
//     x = token id          y = count (occurrences of the root-to-node path)
//     z = index of the first entry of this node's own child run
//     w = number of children (low 24 bits) | RUN_STATIC (bit 31) | RUN_HAS_TOP (bit 30)
// A child run is a contiguous array of entries sorted by token id, so one
// 16-byte load per child yields everything Eq. 1 needs (token, count) plus the
// way down.  A run with n children built online has room for pow2ceil(n)
// entries; a run laid down by the offline build is an exact fit (RUN_STATIC)
// and moves to a roomier place on its first insert.  Depth-1 nodes are found
// through a direct table root[token] -> entry index (-1: absent), so the root
// needs no run of its own.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "suffixspec.h"

#define SD_MAX_DEPTH 32
#define SD_MAX_SPEC 64
#define RUN_STATIC 0x80000000u
#define RUN_COUNT_MASK 0x00FFFFFFu
#define RUN_UNKNOWN 0xFFFFFFFFu
// A long child run laid down by the offline build is preceded by a TOP BLOCK: one header entry
// {sum of the children's counts (lo, hi), number of top entries, 0} and copies of the 64
// children with the largest counts (then smallest tokens), best first.  Only those can ever
// enter a speculation tree of at most 64 nodes, so expanding such a node reads 1 KB instead
// of the whole run.  The flag is dropped by the first online update that touches the run.
#define RUN_HAS_TOP 0x40000000u
#define SD_TOP_MIN 128            // runs longer than this get a top block
#define SD_TOP_BLOCK 65           // entries of a top block
#define SD_OCC_LANES 32           // a per-request match node with at most this many occurrences is expanded a lane per occurrence

struct GlobalState {          // device-resident bookkeeping of the global tree
    int32_t used;             // entries handed out
    int32_t live;             // live nodes
    int32_t status;           // SD_STATUS_GLOBAL_FULL or 0
    int32_t epoch;            // grows whenever an online insert changed the tree
    long long tokens;         // tokens inserted
};

struct SlotState {            // device-resident bookkeeping of one request slot
    int32_t len;              // context length t
    int32_t used;             // entries handed out of the slot pool
    int32_t live;             // live nodes
    int32_t status;           // SD_STATUS_*
    int32_t active[SD_MAX_DEPTH];   // active[d-1]: entry of the node for the last d tokens
    int32_t room[SD_MAX_DEPTH];     // free entries reserved right behind that node for its chain
    int32_t run_cb[SD_MAX_DEPTH];   // that node's child run: first entry ...
    uint32_t run_w[SD_MAX_DEPTH];   // ... and its w field (count | flags); RUN_UNKNOWN: read the entry
    // Match nodes of this request in the GLOBAL tree, kept from the last sd_speculate so that
    // the next one only descends the tokens appended since (a cache: losing it costs a full walk).
    int32_t gen;              // grows when the slot is reset
    int32_t g_gen;            // value of gen the cache was taken at
    int32_t g_epoch;          // global epoch the cache was taken at
    int32_t g_len;            // context length the cache was taken at
    int32_t g_depths;         // depths 1..g_depths are cached
    int32_t g_node[SD_MAX_DEPTH];   // g_node[d-1]: global node of the last d tokens, -1 none
};

struct sd_workspace {         // grow-only device buffers, reused call after call
    void* ptr[48];
    long long bytes[48];
};

struct sd_store {
    int32_t V, D, R, T, M;
    int32_t device;           // the CUDA device that owns the store
    // global tree
    int4* g_ent;
    long long g_cap;
    int32_t* g_root;          // [V]
    GlobalState* g_state;
    // per-request trees
    int4* s_ent;              // [R][spn]
    long long spn;
    int32_t* s_root;          // [R][V]
    int32_t* s_text;          // [R][T]
    SlotState* s_state;       // [R]
    // per-job records of the two-kernel form (sd_speculate_noalloc points them at its fixed array;
    // the store itself allocates none): one record per (request, tree, p) job
    double* j_score;          // [R*2*D]
    int32_t* j_n;             // [R*2*D]
    int32_t* j_tok;           // [R*2*D][M]
    int32_t* j_par;           // [R*2*D][M]
    long long device_bytes;
    struct sd_workspace* ws;  // HOST: temporaries of sd_build_requests, kept between calls
    // HOST: sd_append runs the insert into the global tree beside the appends to the request trees
    // (they share nothing), on this stream, forked from and joined to the caller's stream
    cudaStream_t aux;
    cudaEvent_t ev_fork, ev_join;
};

__host__ __device__ inline uint32_t sd_pow2ceil(uint32_t n) {
#ifdef __CUDA_ARCH__
    return n <= 1u ? 1u : 1u << (32 - __clz((int)(n - 1u)));
#else
    uint32_t c = 1;
    while (c < n) c <<= 1;
    return c;
#endif
}

// Room of a child run that currently holds n children.
__host__ __device__ inline uint32_t sd_run_capacity(uint32_t w) {
    uint32_t n = w & RUN_COUNT_MASK;
    if (n == 0) return 0;
    return (w & RUN_STATIC) ? n : sd_pow2ceil(n);
}

#define SD_CUDA_OK(expr)                                   \
    do {                                                   \
        cudaError_t _e = (expr);                           \
        if (_e != cudaSuccess) return SD_ERR_CUDA;         \
    } while (0)

// Every entry point refuses a store that lives on another device than the current one.
#define SD_CHECK_DEVICE(s)                                                   \
    do {                                                                     \
        int _dev = -1;                                                       \
        if (cudaGetDevice(&_dev) != cudaSuccess) return SD_ERR_CUDA;         \
        if (_dev != (s)->device) return SD_ERR_INVALID_ARG;                  \
    } while (0)
