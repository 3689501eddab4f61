// Internal definitions shared by the libcstr translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "cstr.h"

#define CSTR_DEAD (-1)
#define CSTR_HOST_SLICES 8       // row slices of cstr_step_host

// Set the calling thread's error message (printf-style) and return `code`.
int cstr_fail(int code, const char *fmt, ...);

// CSTR_OK if `handle_device` is the current CUDA device, else CSTR_ERR_DEVICE
// (or CSTR_ERR_CUDA) with a message naming `what`.
int cstr_check_device(int handle_device, const char *what);

#define CSTR_CUDA_TRY(expr)                                                              \
    do {                                                                                 \
        cudaError_t e_ = (expr);                                                         \
        if (e_ != cudaSuccess)                                                           \
            return cstr_fail(e_ == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM            \
                                                             : CSTR_ERR_CUDA,            \
                             "%s failed: %s", #expr, cudaGetErrorString(e_));            \
    } while (0)

// Checking build (-DCSTR_BOUNDS_CHECK): kernels compare every index they form
// into a table, vocabulary or logits array with the array's extent before the
// access.  A violation is counted in a 4-word record on the device (count,
// then site / index / extent of the first one) and the access is skipped; no
// trap, no assert.  In the release build CSTR_INB is the constant true and
// the checks vanish.
#define CSTR_SITE_BUILD_TT 1        // builder: DFA table lookup
#define CSTR_SITE_BUILD_NEXT 2      // builder: store into next
#define CSTR_SITE_BUILD_MASKT 3     // builder: ballot words
#define CSTR_SITE_BUILD_VOCAB 4     // builder: descriptors, offsets, bytes
#define CSTR_SITE_BUILD_STACK 5     // builder: shared-memory stack / staged table
#define CSTR_SITE_TRANSPOSE 6       // mask transpose: maskT read, mask write
#define CSTR_SITE_GROUP 7           // duplicate-column pass scratch
#define CSTR_SITE_EXPAND 8          // duplicate-column pass: row copies
#define CSTR_SITE_TERMINALS 9       // terminal-label post-pass
#define CSTR_SITE_STEP_LOGITS 10    // step: logits / noise / masked output
#define CSTR_SITE_STEP_MASK 11      // step: mask words
#define CSTR_SITE_STEP_NEXT 12      // step: next-state gather, accept flag
#define CSTR_SITE_STEP_ROW 13       // step: per-row arrays and scratch
#define CSTR_SITE_DOWNLOAD 14       // table download decode
#define CSTR_SITE_PDA 15            // push-down kernels
#ifdef CSTR_BOUNDS_CHECK
// Device address of the current device's record (allocated on first use), or null.
unsigned long long *cstr_oob_record();
__device__ __forceinline__ bool cstr_in_bounds(unsigned long long *rec, long long idx,
                                               long long extent, int site)
{
    if (idx >= 0 && idx < extent)
        return true;
    if (rec && atomicAdd(rec, 1ull) == 0ull) {
        rec[1] = (unsigned long long)site;
        rec[2] = (unsigned long long)idx;
        rec[3] = (unsigned long long)extent;
    }
    return false;
}
#define CSTR_INB(rec, idx, extent, site) \
    cstr_in_bounds((rec), (long long)(idx), (long long)(extent), (site))
#define CSTR_OOB_RECORD() cstr_oob_record()
#else
#define CSTR_INB(rec, idx, extent, site) (true)
#define CSTR_OOB_RECORD() ((unsigned long long *)nullptr)
#endif

// State ids inside the builder's tables are permuted within blocks of 256:
// state 256 b + 8 l + j sits at slot 256 b + 32 j + l.  A warp whose lane l
// owns the 8 consecutive states 8 l .. 8 l + 7 then reads 32 consecutive slots
// per lookup round (no shared-memory bank conflicts) as long as the walk keeps
// neighbouring states neighbours, which counters and literal chains do.
#define CSTR_PERM(s) (((s) & ~255) | (((s) & 7) << 5) | (((s) >> 3) & 31))
#define CSTR_UNPERM(v) (((v) & ~255) | (((v) & 31) << 3) | (((v) >> 5) & 7))

// Byte DFA as the builder reads it: bytes that no state tells apart share a
// class, and the table is stored class-major ("transposed") in permuted slots,
// holding permuted targets, with a dead sink (state n_states) that maps to
// itself, so that a walk needs no "is it dead" branch:
//     tt[c][PERM(s)] = code(target of s on class c, or n_states),
//     code(t) = PERM(t) * sizeof(entry): the byte offset of t's slot in a row,
// for s in [0, row), row = n_states + 1 rounded up to 256.
struct cstr_dfa {
    int device;
    int32_t n_states;
    int32_t start;
    int wide;            // 0: int16 entries (n_states + 1 <= 32767), 1: int32 entries
    int32_t n_classes;   // 1..256
    int sparse;          // most states allow few bytes: the builder prunes dead subtrees
    int32_t n_many;      // sparse automata: states that allow many bytes (numbered first)
    // Internal state numbering (null = identity).  For sparse automata the few
    // states that allow most bytes (free text inside a string, say) are numbered
    // first, so that they share warps with each other and the many picky
    // states fill warps that die quickly along the vocabulary trie.  Every
    // table the builder reads or writes (tt, next, the ballot rows) is indexed
    // by internal ids; the mask rows, the accept flags and the ABI use the
    // caller's ids.  rank[q] = internal id of state q, unrank = its inverse,
    // both with the sink n_states mapped to itself.
    int32_t *rank;       // DEVICE [n_states + 1] or null
    int32_t *unrank;     // DEVICE [n_states + 1] or null
    int32_t *rank_host;  // HOST copy of rank (malloc) or null
    int64_t row;         // entries per class row (n_states + 1, rounded up to 256)
    void *tt;            // DEVICE [n_classes][row]
    uint8_t *cls;        // DEVICE [256] byte -> class
    uint8_t *accept;     // DEVICE [n_states]
    // terminal-label edges, kept only for the states that have any
    int32_t n_labels;
    int32_t n_term_states;
    int32_t *tstate;     // DEVICE [n_term_states] state ids
    uint32_t *tset;      // DEVICE [n_term_states] labels with an edge (bit set)
    uint32_t *ttarget;   // DEVICE [n_term_states][n_labels] target codes
};

// Vocabulary as the builder reads it: tokens in lexicographic (trie depth-first)
// order, each with the length of the prefix it shares with its predecessor, so
// that a walk resumes at the shared depth instead of at the root.
//   desc[i] = { token id, length | shared_prefix << 24, first 8 bytes after the
//               shared prefix (little endian in z, w) }
// The shared prefix is clipped to CSTR_STACK_DEPTH.  Raw bytes / offsets serve
// walks that start at the root and suffixes longer than 8 bytes.
#define CSTR_STACK_DEPTH 4
struct cstr_vocab {
    int device;
    int32_t V;
    int64_t total_bytes;
    uint8_t *bytes;    // DEVICE [total_bytes + 16]
    uint32_t *off;     // DEVICE [V + 1]
    uint4 *desc;       // DEVICE [V], sorted order
    uint32_t *pre4;    // DEVICE [V], sorted order: the token's first 4 bytes (little endian, 0-padded)
    uint32_t max_len;
    int32_t n_labels;  // terminal labels with a token set (0 = none attached)
    uint32_t *by_len;  // DEVICE [V] token ids ordered by length (then id): warps of equal-length tokens
    uint32_t *tsets;   // DEVICE [V] bit t: token belongs to label t's set
};

// Token table.  next is token-major: next[v][q] (a step reads one entry per
// row; the builder writes whole state segments); entries are the unsigned
// codes the builder walks with (CSTR_PERM(state) << code_shift), "no edge"
// being the code of the sink state n_states.  mask is state-major
// as the step streams it.  maskT is the builder's intermediate: per token one
// word per block of 32 states, transposed into mask by a second kernel.
struct cstr_table {
    int device;
    const cstr_vocab *vocab;
    cstr_vocab *owned_vocab;   // non-null when created by cstr_build_token_table
    int32_t max_states;
    int32_t V, W;
    int64_t lds;       // entries per token row of next (max_states rounded up to 256)
    int64_t ldw;       // words per state row of mask (W rounded up to 32), padding zero
    int64_t ldb;       // words per token row of maskT (state blocks rounded up to 8)
    int wide;          // capacity dtype of next: 0 int16, 1 int32
    void *next;        // DEVICE [V][lds]
    uint32_t *mask;    // DEVICE [max_states][ldw]
    uint32_t *maskT;   // DEVICE [V][ldb]
    uint8_t *accept;   // DEVICE [max_states]
    int32_t n_states;  // of the automaton currently held (0 = not built)
    int32_t start;
    int32_t eos_id;
    int32_t code_shift; // next entries are CSTR_PERM(state) << code_shift (1: 16-bit DFA, 2: 32-bit)
    // Status word of the builder's bulk-copy pipeline: non-zero once a bounded wait
    // of a build gave up (never expected; reported by cstr_table_download).
    unsigned int *build_status;    // DEVICE [1]
    // internal state numbering of the automaton currently held (see cstr_dfa)
    int renumbered;     // 0: identity, rank / unrank unused
    int32_t *rank;      // DEVICE [max_states + 1]
    int32_t *unrank;    // DEVICE [max_states + 1]
    // Scratch of the builder's duplicate-column pass (tokens that read as the same
    // string of byte classes share one walk): an open-addressing table keyed by a
    // 64-bit hash of the class string, each sorted token's representative, the
    // representatives' own trie-ordered descriptor list and its length.
    uint32_t group_slots;          // power of two >= 4 V
    unsigned long long *group_key; // DEVICE [group_slots]
    uint32_t *group_min;           // DEVICE [group_slots] smallest sorted index of the group
    uint32_t *group_rep;           // DEVICE [V] representative's sorted index, per sorted index
    uint32_t *group_reptok;        // DEVICE [V] representative's token id, per token id
    uint4 *group_desc;             // DEVICE [V] descriptors of the representatives, in order
    int32_t *group_count;          // DEVICE [1] number of representatives
    uint32_t *group_uniq;          // DEVICE [V] sorted indices of the representatives, in order
    int32_t *group_blk;            // DEVICE [ceil(V / 1024)] representatives per 1,024 sorted tokens
};

struct cstr_workspace {
    int device;
    int32_t max_batch;
    unsigned long long *cell;      // DEVICE [max_batch] packed (value, index) running maxima
    unsigned int *ticket;          // DEVICE [max_batch] arrival counters
    unsigned long long *counters;  // DEVICE [2] bad-state rows, empty-mask rows
    // cstr_step_host only (created on its first use): a copy stream and one event
    // per slice of rows, so that uploads run ahead of the step kernels
    cudaStream_t copy_stream;      // host -> device
    cudaStream_t down_stream;      // device -> host (penalised logits, when asked for)
    cudaEvent_t slice_ready[CSTR_HOST_SLICES];
    cudaEvent_t slice_done[CSTR_HOST_SLICES];
    cudaEvent_t inputs_free;
    int host_ready;
};

// Byte-level PDA as the kernels read it.  act[(q * NT + t) * 256 + byte] is the
// index of the edge taken from state q on `byte` when the top of the stack is
// t, for t = a symbol, n_symbols ("stack empty") or n_symbols + 1 ("top not
// known": only edges that pop nothing qualify; CSTR_PDA_NEEDCTX if the answer
// depends on the symbol), or CSTR_PDA_NONE.
// edge[j] = { target, push0 | push1 << 8 | push2 << 16 | npush << 24 | pop << 28 }.
#define CSTR_PDA_NONE 0xffffffffu
#define CSTR_PDA_NEEDCTX 0xfffffffeu
struct cstr_pda_view {
    const uint32_t *act;
    const int2 *edge;
    int NT;
    int n_symbols;
    // extents, for the checking build's range checks
    long long act_len;             // entries of act
    int n_edges;
    unsigned long long *oob;       // bounds record, null in the release build
};

// What the step kernel needs to traverse an edge of the token-level PDA.
struct cstr_pda_advance {
    cstr_pda_view P;
    const uint8_t *accept;         // DEVICE [n_states]
    const uint8_t *vbytes;         // DEVICE vocabulary bytes
    const uint32_t *voff;          // DEVICE [V + 1]
    int32_t n_states, eos_id, cap;
    // situation before the step (read) and after it (written); the two sets may
    // be the same arrays (in-place update) or different ones (state history)
    const int32_t *states_in, *stacks_in, *depths_in;
    int32_t *states, *stacks, *depths;   // DEVICE [batch], [batch][cap], [batch]
    uint8_t *accept_out;           // DEVICE [batch] or null
    unsigned long long *counters;  // DEVICE [3]: bad rows, rows without a token, overflows
};

struct cstr_pda {
    int device;
    int32_t n_states, n_symbols, start, n_edges;
    int32_t NT;          // n_symbols + 2
    int32_t max_push;    // largest number of symbols one edge pushes
    uint32_t *act;       // DEVICE [n_states][NT][256]
    int2 *edge;          // DEVICE [n_edges]
    uint8_t *accept;     // DEVICE [n_states]
};

// Token-level PDA: one row of allowed-token words and one of "depends on deeper
// symbols" words per situation cfg = q * (n_symbols + 1) + top (top = n_symbols
// for the empty stack); ndeep[cfg] = number of bits set in deep[cfg].
struct cstr_pda_table {
    int device;
    const cstr_pda *pda;
    const cstr_vocab *vocab;
    int32_t V, W;
    int64_t ldw;         // words per row (W rounded up to 32), padding zero
    int32_t n_cfg;
    int32_t eos_id;
    uint32_t *mask;      // DEVICE [n_cfg][ldw]
    uint32_t *deep;      // DEVICE [n_cfg][ldw]
    uint32_t *ndeep;     // DEVICE [n_cfg]
    // builder scratch, per state: tokens allowed whatever the stack holds, and
    // tokens whose walk looks at the top of the stack
    uint32_t *base;      // DEVICE [n_states][ldw]
    uint32_t *need;      // DEVICE [n_states][ldw]
};

struct cstr_pda_workspace {
    int device;
    int32_t max_batch;
    int64_t ldw;
    unsigned long long *cell;      // DEVICE [max_batch]
    unsigned int *ticket;          // DEVICE [max_batch]
    unsigned long long *counters;  // DEVICE [4]: step's two (unused), then bad / empty / overflow
    const uint32_t **row_mask;     // DEVICE [max_batch]
    uint32_t *row_buf;             // DEVICE [max_batch][ldw]
};

// Kernel launchers (defined in cstr_build.cu / cstr_step.cu).
// dense_walk: every token walked from its first byte (no shared prefixes): the baseline
int cstr_launch_build(cstr_table *table, const cstr_dfa *dfa, cudaStream_t stream,
                      bool dense_walk = false);

struct cstr_step_args {
    const cstr_table *tables[CSTR_MAX_TABLES];
    int32_t n_tables;
    const int32_t *row_table;
    const void *logits;
    int32_t dtype;
    int64_t ld;
    const float *noise;
    const int32_t *states;
    int32_t *states_out;           // may equal states (in-place update)
    int32_t *tokens_out;
    void *masked_out;
    uint8_t *accept_out;
    int32_t batch;
    // scratch, zero on entry and left zero by the kernel (see cstr_step.cu)
    unsigned long long *cell;      // DEVICE [batch]
    unsigned int *ticket;          // DEVICE [batch]
    unsigned long long *counters;  // DEVICE [2]
    int device;
    // Push-down mode: when pda is non-null the kernel takes row r's allowed-token
    // words from row_mask[r] (null = inactive row), needs no tables, and the last
    // CTA of a row traverses the selected token's edge of the token-level PDA
    // (state, stack, depth, accept flag, counters: see cstr_pda_advance).
    const struct cstr_pda_advance *pda;   // HOST
    const uint32_t *const *row_mask;      // DEVICE [batch]
    int32_t V;                            // vocabulary size  (push-down mode only)
    int64_t ldw;                          // words readable behind every row pointer
};
int cstr_launch_step(const cstr_step_args &a, cudaStream_t stream);
int cstr_launch_accept(const int32_t *draft, const int32_t *tgt_tok, const int32_t *tgt_state,
                       int32_t k, int32_t batch, int32_t *n_accepted, int32_t *out_tokens,
                       int32_t *states, cudaStream_t stream);
