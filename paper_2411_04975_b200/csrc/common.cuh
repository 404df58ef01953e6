// Shared declarations of the suffixspec CUDA library (sm_100a).
//
// Global tree: node storage.  A tree node is a 16-byte ENTRY that lives inside its parent's
// child run:
//     x = token id          y = count (occurrences of the root-to-node path)
//     z = index of the first entry of this node's own child run
//     w = number of children (low 24 bits) | flags (RUN_STATIC, RUN_HAS_TOP, NODE_TOUCHED)
// A child run is a contiguous array of entries sorted by token id, so one
// 16-byte load per child yields everything Eq. 1 needs (token, count) plus the
// way down.  A run with n children built online has room for pow2ceil(n)
// entries; a run laid down by the offline build is an exact fit (RUN_STATIC)
// and moves to a roomier place on its first insert.  Depth-1 nodes are found
// through a direct table root[token] -> entry index (-1: absent), so the root
// needs no run of its own.
//
// Beside the entries the store keeps what the offline build sorted: the corpus text, its suffix
// order and, per child run, the place of the run's owner in that order.  A node that no online
// insert has touched is then also a RANGE of the suffix order: its occurrences are listed there,
// and the tokens around each occurrence are plain text (see occurrence mode in speculate.cu).
//
// Per-request trees are IMPLICIT: the tree over a request's text x_{1:t} is the set of its
// substrings of at most D tokens with their numbers of occurrences.  The store keeps the text
// and the order of its suffixes (suffix_order.cuh): a node is a range of that order, its count
// the range's size, its children the runs of equal next tokens.  Appending a token is writing
// it and giving the few suffixes it changes their new places; a thread block holds text and
// order in shared memory while it works on a request.
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
// Set on every node an online insert created or counted up: its count (and what lies below it)
// is no longer what the suffix order of the offline build says.
#define NODE_TOUCHED 0x20000000u
#define SD_TOP_MIN 128            // runs longer than this get a top block
#define SD_TOP_BLOCK 65           // entries of a top block
#define SD_OCC_LANES 32           // a node with at most this many occurrences is expanded a lane per occurrence
#define SD_OCC_BASE 64            // a global match node with at most this many occurrences stands in for all longer patterns

struct GlobalState {          // device-resident bookkeeping of the global tree
    int32_t used;             // entries handed out
    int32_t live;             // live nodes
    int32_t status;           // SD_STATUS_GLOBAL_FULL or 0
    int32_t epoch;            // grows whenever an online insert changed the tree
    long long tokens;         // tokens inserted
};

struct SlotState {            // device-resident bookkeeping of one request slot
    int32_t len;              // context length t
    int32_t status;           // SD_STATUS_*
    int32_t gen;              // grows when the slot is reset
    // Match nodes of this request in the GLOBAL tree, kept from the last speculation so that the
    // next one only descends the tokens appended since (a cache: losing it costs walks from the root).
    int32_t g_gen;            // value of gen the cache was taken at
    int32_t g_epoch;          // global epoch the cache was taken at
    int32_t g_len;            // context length the cache was taken at
    int32_t g_depths;         // pattern lengths 1..g_depths are cached
    int32_t sa_buf;           // which of the slot's two suffix-order arrays is the current one
    int32_t g_node[SD_MAX_DEPTH];   // g_node[d-1]: global node of the last d tokens, -1 none
};

struct sd_store {
    int32_t V, D, R, T, M;
    int32_t Tp;               // row stride of s_text and of the occurrence scratch (T rounded up to 4)
    int32_t device;           // the CUDA device that owns the store
    // global tree
    int4* g_ent;
    long long g_cap;
    int32_t* g_root;          // [V]
    GlobalState* g_state;
    // what the offline build sorted (N0 tokens; nothing of it changes afterwards)
    long long N0;
    long long static_entries; // entries laid down by the offline build: g_lo covers [0, static_entries)
    int32_t* g_text;          // [N0] corpus
    uint32_t* g_sa;           // [N0] suffix order: text position of the j-th smallest suffix
    uint8_t* g_len;           // [N0] by rank: tokens of that suffix inside its sequence, capped at D
    uint8_t* g_back;          // [N0] by text position: tokens before it inside its sequence, capped at D
    int32_t* g_lo;            // [static_entries] by first entry of a child run: rank of the owner's first suffix
    // per-request trees: the texts
    int32_t* s_text;          // [R][Tp]
    int32_t* s_sa;            // [2][R][Tp] suffix order of each text (suffix_order.cuh); an update reads one
                              // array and writes the other, SlotState.sa_buf says which is current
    SlotState* s_state;       // [R]
    int32_t* occ_scratch;     // [R][Tp]: work buffer for the suffix order of a text too long for shared memory
    // staging of sd_build_requests' host arrays
    int32_t* stage_slot;      // [R]
    int64_t* stage_off;       // [R + 1]
    long long device_bytes;
    // HOST: sd_append runs the insert into the global tree beside the appends to the request texts
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
