// Internal definitions shared by the libcstr translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "cstr.h"

#define CSTR_DEAD (-1)

// Set the calling thread's error message (printf-style) and return `code`.
int cstr_fail(int code, const char *fmt, ...);

#define CSTR_CUDA_TRY(expr)                                                              \
    do {                                                                                 \
        cudaError_t e_ = (expr);                                                         \
        if (e_ != cudaSuccess)                                                           \
            return cstr_fail(e_ == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM            \
                                                             : CSTR_ERR_CUDA,            \
                             "%s failed: %s", #expr, cudaGetErrorString(e_));            \
    } while (0)

struct cstr_dfa {
    int device;
    int32_t n_states;
    int32_t start;
    int wide;          // 0: int16 entries, 1: int32 entries
    void *trans;       // DEVICE [n_states][256]
    uint8_t *accept;   // DEVICE [n_states]
};

// Vocabulary as the builder reads it: the first 16 bytes of every token packed
// in one 16-byte record (zero padded), its length, and the raw bytes/offsets
// for the rare longer token.
struct cstr_vocab {
    int device;
    int32_t V;
    int64_t total_bytes;
    uint8_t *bytes;    // DEVICE [total_bytes + 16]
    uint32_t *off;     // DEVICE [V + 1]
    uint4 *head;       // DEVICE [V]    first 16 bytes
    uint32_t *len;     // DEVICE [V]
    uint32_t max_len;
};

struct cstr_table {
    int device;
    const cstr_vocab *vocab;
    cstr_vocab *owned_vocab;   // non-null when created by cstr_build_token_table
    int32_t max_states;
    int32_t V, W;
    int64_t ldn;       // elements per row of next (V rounded up to 64)
    int64_t ldw;       // words per row of mask (W rounded up to 32), padding zero
    int wide;          // capacity dtype of next: 0 int16, 1 int32
    void *next;        // DEVICE [max_states][ldn]
    uint32_t *mask;    // DEVICE [max_states][ldw]
    uint8_t *accept;   // DEVICE [max_states]
    int32_t n_states;  // of the automaton currently held (0 = not built)
    int32_t start;
    int32_t eos_id;
};

struct cstr_workspace {
    int device;
    int32_t max_batch;
    unsigned long long *cell;      // DEVICE [max_batch] packed (value, index) running maxima
    unsigned int *ticket;          // DEVICE [max_batch] arrival counters
    unsigned long long *counters;  // DEVICE [2] bad-state rows, empty-mask rows
};

// Kernel launchers (defined in cstr_build.cu / cstr_step.cu).
int cstr_launch_build(cstr_table *table, const cstr_dfa *dfa, cudaStream_t stream);

struct cstr_step_args {
    const cstr_table *tables[CSTR_MAX_TABLES];
    int32_t n_tables;
    const int32_t *row_table;
    const void *logits;
    int32_t dtype;
    int64_t ld;
    const float *noise;
    int32_t *states;
    int32_t *tokens_out;
    void *masked_out;
    uint8_t *accept_out;
    int32_t batch;
    // scratch, zero on entry and left zero by the kernel (see cstr_step.cu)
    unsigned long long *cell;      // DEVICE [batch]
    unsigned int *ticket;          // DEVICE [batch]
    unsigned long long *counters;  // DEVICE [2]
    int device;
};
int cstr_launch_step(const cstr_step_args &a, cudaStream_t stream);
