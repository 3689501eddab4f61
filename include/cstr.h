/*
 * libcstr - regular-language constraints for batched LM decoding on one GPU.
 *
 * The library holds the data-parallel part of the automata-based constraint
 * method of "Automata-based constraints for language model decoding":
 *
 *   1. the token-level automaton: the composition of a character (byte) DFA
 *      with the vocabulary's detokenizer, emitted densely as
 *          next[q][v] = delta*(q, bytes(v))      (-1 = no edge)
 *          mask[q] bit v = (next[q][v] != -1)
 *      for every DFA state q and vocabulary token v;
 *   2. the per-step recipe: mask from the current state, penalise the logits
 *      with -infinity, select a token, advance the state - for a whole batch.
 *
 * Conventions
 *   - Every function returns 0 (CSTR_OK) or a negative CSTR_ERR_* code and
 *     never throws, aborts or traps; cstr_last_error() gives a message for the
 *     calling thread's last failure.
 *   - "HOST" / "DEVICE" says where a pointer must point.  The caller owns all
 *     such arrays; the library owns what is behind its opaque handles and frees
 *     it in the matching cstr_free_*.  Handles are bound to the CUDA device
 *     that was current when they were created; that device must be current in
 *     later calls.
 *   - cuda_stream is a cudaStream_t passed as void* (NULL = default stream).
 *   - S = DFA states, V = vocabulary size, W = ceil(V / 32) mask words.
 */
#ifndef CSTR_H
#define CSTR_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CSTR_OK 0
#define CSTR_ERR_NULL (-1)      /* a required pointer was NULL                        */
#define CSTR_ERR_ARG (-2)       /* a size / index argument is out of range            */
#define CSTR_ERR_DFA (-3)       /* transition target outside [-1, S)                  */
#define CSTR_ERR_VOCAB (-4)     /* offsets decreasing, negative or too large          */
#define CSTR_ERR_DTYPE (-5)     /* unknown logits dtype                               */
#define CSTR_ERR_SHAPE (-6)     /* ld < V, tables with different V, capacity exceeded */
#define CSTR_ERR_CUDA (-7)      /* a CUDA runtime call failed                         */
#define CSTR_ERR_NOMEM (-8)     /* host or device allocation failed                   */
#define CSTR_ERR_DEVICE (-9)    /* handle belongs to another CUDA device              */
#define CSTR_ERR_PDA (-10)      /* byte PDA malformed, non-deterministic or over a limit */

#define CSTR_F32 0              /* logits are IEEE fp32                               */
#define CSTR_BF16 1             /* logits are bfloat16                                */

#define CSTR_MAX_TABLES 16      /* tables one cstr_step call can mix                  */

typedef struct cstr_dfa cstr_dfa_t;             /* device copy of a byte-level DFA            */
typedef struct cstr_vocab cstr_vocab_t;         /* device copy of a vocabulary                */
typedef struct cstr_table cstr_table_t;         /* device mask[S][W] + next[S][V]             */
typedef struct cstr_workspace cstr_workspace_t; /* per-stream scratch of cstr_step            */
typedef struct cstr_pda cstr_pda_t;             /* device copy of a byte-level PDA            */
typedef struct cstr_pda_table cstr_pda_table_t; /* token-level PDA: masks per (state, top)    */
typedef struct cstr_pda_workspace cstr_pda_workspace_t; /* per-stream scratch of cstr_pda_step */

/* ------------------------------------------------------------------ DFA */

/*
 * Load a deterministic byte-level FSA (Section 2.1: an FSA (Sigma, Q, I, F, E)
 * that is deterministic has no epsilon edge and at most one edge per state and
 * symbol, so it is a table).  Sigma is the 256 byte values.
 *   trans        HOST  int32 [n_states][256], target state or -1 (no edge)
 *   accept       HOST  uint8 [n_states], non-zero = final state
 *   n_states     1 .. 4,000,000;  start_state in [0, n_states)
 * Validates every target, merges bytes that no state tells apart into
 * classes, and copies the class-major table to the device (16-bit entries up
 * to 32766 states, else 32-bit); returns the handle in *out.
 * Synchronous; allocates device memory.  Each host thread keeps the device
 * scratch of its last load (the raw table, at most 64 MB) for the next one
 * and frees it when the thread ends.
 */
int cstr_load_dfa(const int32_t *trans, const uint8_t *accept, int32_t n_states,
                  int32_t start_state, cstr_dfa_t **out);
void cstr_free_dfa(cstr_dfa_t *dfa);

/*
 * As cstr_load_dfa, for an automaton that also has edges labelled with
 * terminal labels (Section 2.5.1, "Wildcard matching"): symbols outside the
 * byte alphabet, each standing for a pre-computed set of tokens, written
 * (?P<NAME>) in a regex.
 *   term_trans   HOST  int32 [n_states][n_labels], target state or -1
 *   n_labels     0..32; label t is bit t of the token sets given to
 *                cstr_vocab_set_token_sets
 * In the built table a state's terminal edges allow every token of their
 * labels' sets on top of the ordinary tokens (whole sets at once); a selected
 * token follows its ordinary edge if it has one, else the terminal edge of the
 * lowest label whose set holds it (the paper's precedence heuristic).
 */
int cstr_load_dfa_terminals(const int32_t *trans, const int32_t *term_trans, int32_t n_labels,
                            const uint8_t *accept, int32_t n_states, int32_t start_state,
                            cstr_dfa_t **out);

/* ---------------------------------------------------------------- vocab */

/*
 * Load a vocabulary: token v detokenizes to vocab_bytes[offsets[v] ..
 * offsets[v+1]) (App. B.1: each token has one character sequence d(v); the
 * detokenization of a token sequence is the concatenation).  This is the
 * vocabulary-specific half of the method, prepared once per LM like the
 * detokenizing transducer T_V of Algorithm 1 (Section 2.4 notes that T_V
 * depends only on the vocabulary and can be built ahead of time).
 *   vocab_bytes  HOST  uint8 [offsets[vocab_size]]
 *   offsets      HOST  int64 [vocab_size + 1], offsets[0] == 0, non-decreasing,
 *                total below 2^31
 * Duplicate strings are allowed (each id gets its own column).  A token of
 * length 0 never has an edge.  Synchronous; allocates device memory.
 */
int cstr_load_vocab(const uint8_t *vocab_bytes, const int64_t *offsets, int32_t vocab_size,
                    cstr_vocab_t **out);
void cstr_free_vocab(cstr_vocab_t *vocab);

/*
 * Attach the token sets of the terminal labels to a vocabulary (Section 2.5.1:
 * every terminal label stands for a mask of tokens computed ahead of time,
 * e.g. the newline-free tokens for PARAGRAPH_TOKEN).  Prepared once per LM.
 *   token_sets   HOST  uint32 [vocab_size]; bit t set iff the token belongs to
 *                the set of label t
 *   n_labels     1..32
 * Replaces any sets attached before.  Synchronous; allocates device memory.
 * Tokens of length 0 never match a label.
 */
int cstr_vocab_set_token_sets(cstr_vocab_t *vocab, const uint32_t *token_sets, int32_t n_labels);

/* ---------------------------------------------------------------- table */

/*
 * Allocate an empty token table able to hold up to max_states states over
 * `vocab`.  `vocab` must outlive every cstr_table_build on this table.
 */
int cstr_table_create(const cstr_vocab_t *vocab, int32_t max_states, cstr_table_t **out);

/*
 * Build the token-level automaton A_{R o V} = Determinize(A_R o T_V) of
 * Algorithm 2 in its dense form (Theorem 2 fixes its meaning: a token sequence
 * is accepted iff its detokenization is accepted by the DFA):
 *     next[q][v] = state reached from q by reading bytes(v), -1 as soon as a
 *                  byte has no edge or if the token is empty
 *     mask[q] word v/32 bit v%32 (LSB first) = next[q][v] != -1; unused high
 *                  bits of the last word are 0
 * If eos_id >= 0, that token's bytes are ignored: it is allowed exactly in
 * accepting states and leads to -1 ("finished").
 * A DFA loaded with terminal labels needs a vocabulary with token sets for at
 * least as many labels (else CSTR_ERR_SHAPE); its terminal edges are merged
 * into mask and next as described at cstr_load_dfa_terminals.
 * Only enqueues kernels on cuda_stream: no allocation, no host synchronisation.
 * The table may be rebuilt any number of times (dfa->n_states <= max_states);
 * it must not be in use by a cstr_step that has not completed.
 */
int cstr_table_build(cstr_table_t *table, const cstr_dfa_t *dfa, int32_t eos_id,
                     void *cuda_stream);

/*
 * The same table as cstr_table_build, computed the plain way: every token is
 * walked from its first byte for every state, as if the detokenizing
 * transducer were Algorithm 1's one chain per token with no prefix shared
 * between tokens (Section 2.3 describes the compact, trie-shaped T_V that
 * cstr_table_build walks instead).  Same arguments, same results, slower; it
 * exists so that the saving of the trie walk can be measured on any
 * constraint.
 */
int cstr_table_build_dense(cstr_table_t *table, const cstr_dfa_t *dfa, int32_t eos_id,
                           void *cuda_stream);

/*
 * One-call form: load the vocabulary from HOST arrays (as cstr_load_vocab),
 * create a table sized for `dfa` and build it.  The table owns its private
 * vocabulary copy.  Allocates; the build itself is enqueued on cuda_stream.
 */
int cstr_build_token_table(const cstr_dfa_t *dfa, const uint8_t *vocab_bytes,
                           const int64_t *offsets, int32_t vocab_size, int32_t eos_id,
                           void *cuda_stream, cstr_table_t **out);

/* Shape of the automaton the table currently holds (any pointer may be NULL). */
int cstr_table_info(const cstr_table_t *table, int32_t *n_states, int32_t *vocab_size,
                    int32_t *mask_words, int32_t *start_state);

/*
 * Copy states [state_lo, state_hi) of a built table to the host in logical
 * form, whatever the device layout is:
 *   mask_host  HOST uint32 [(state_hi-state_lo)][W]      or NULL
 *   next_host  HOST int32  [(state_hi-state_lo)][V]      or NULL   (-1 = no edge)
 * Synchronises cuda_stream first and before it returns.  When next_host is
 * given it allocates (and frees) a device staging buffer of at most 256 MB,
 * decodes slabs of states into it on cuda_stream and copies them down.
 */
int cstr_table_download(const cstr_table_t *table, int32_t state_lo, int32_t state_hi,
                        uint32_t *mask_host, int32_t *next_host, void *cuda_stream);
void cstr_free_table(cstr_table_t *table);

/* ----------------------------------------------------------------- step */

/*
 * Scratch for cstr_step: 16 bytes per row plus status counters, zeroed.  Use
 * one workspace per stream; two steps that may overlap on the GPU must not
 * share one.
 */
int cstr_workspace_create(int32_t max_batch, cstr_workspace_t **out);
void cstr_free_workspace(cstr_workspace_t *ws);

/*
 * One constrained decoding step for `batch` independent rows (Algorithm 2,
 * loop body; the three-step recipe of Section 1), in one kernel:
 *   A      = tokens v with mask bit set for the row's state q
 *   masked = logits where v in A, -infinity elsewhere (allowed entries are bit
 *            copies, NaN payloads and -0 included)
 *   token  = argmax over v in A of fp32(logits[v]) (+ noise[v], one rounded
 *            fp32 addition); equal values: lowest id; NaN never wins; an allowed
 *            -infinity still beats "none"
 *   q      = next[q][token]
 *
 *   tables, n_tables  HOST array of 1..CSTR_MAX_TABLES built tables with equal V
 *   row_table   DEVICE int32 [batch] table index per row, or NULL (all rows: tables[0])
 *   logits      DEVICE [batch][ld] of `dtype`; ld >= V is the row stride in elements
 *   noise       DEVICE float [batch][ld] or NULL (greedy); e.g. Gumbel noise for sampling
 *   states      DEVICE int32 [batch], in/out; all rows of a fresh sequence start
 *               at the table's start state
 *   tokens_out  DEVICE int32 [batch]
 *   masked_out  DEVICE [batch][ld] of `dtype`; columns >= V are not written; may be
 *               the same buffer as logits (exactly equal pointers, in-place)
 *   accept_out  DEVICE uint8 [batch] or NULL: 1 iff the new state is accepting
 * A row whose state is -1 (finished / inactive), out of range, or whose table
 * index is out of range, and a row with no selectable token, get token -1,
 * state -1 and all -infinity; nothing out of bounds is ever touched.
 * Only enqueues work on cuda_stream (no allocation, no host synchronisation).
 * With batch == 0 the per-row pointers may be NULL and nothing is enqueued.
 * The fast path needs logits / masked_out / noise 16-byte aligned with
 * ld * sizeof(element) a multiple of 16; other layouts take a slower kernel.
 */
int cstr_step(const cstr_table_t *const *tables, int32_t n_tables, const int32_t *row_table,
              const void *logits, int32_t dtype, int64_t ld, const float *noise,
              int32_t *states, int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
              int32_t batch, cstr_workspace_t *ws, void *cuda_stream);

/*
 * cstr_step for logits that live in HOST memory (the end-to-end form of the
 * same recipe: Section 1, steps 1-3, for a model whose logits arrive on the
 * host).  The rows are cut into a few slices; each slice is uploaded on an
 * internal copy stream while the step kernels of earlier slices run on
 * cuda_stream, and the tokens (and states) are copied back at the end.
 *   logits_host  HOST  [batch][ld] of `dtype` (pinned memory uploads fastest)
 *   noise_host   HOST  float [batch][ld] or NULL
 *   states       DEVICE int32 [batch], in/out
 *   tokens_host  HOST  int32 [batch]: the selected tokens
 *   states_host  HOST  int32 [batch] or NULL: the new states
 *   logits_dev   DEVICE staging [batch][ld] of `dtype`, overwritten
 *   noise_dev    DEVICE staging float [batch][ld]; NULL exactly when noise_host is NULL
 *   masked_out   DEVICE [batch][ld]: the penalised logits (may equal logits_dev)
 *   masked_host  HOST   [batch][ld] of `dtype`, or NULL: when given, the penalised
 *                logits are also copied there, slice by slice on a third stream
 *                while later slices upload and run
 *   tokens_dev   DEVICE int32 [batch]
 * tables, row_table, accept_out, ws: as in cstr_step.  Synchronous: returns
 * after the results are in tokens_host / states_host / masked_host (it
 * synchronises cuda_stream and its own copy streams, on failure too, so the
 * host buffers are never in use once it has returned).  Allocates no device
 * memory; its first call on a workspace creates two copy streams and a few events.
 */
int cstr_step_host(const cstr_table_t *const *tables, int32_t n_tables, const int32_t *row_table,
                   const void *logits_host, int32_t dtype, int64_t ld, const float *noise_host,
                   int32_t *states, int32_t *tokens_host, int32_t *states_host, void *logits_dev,
                   float *noise_dev, void *masked_out, void *masked_host, int32_t *tokens_dev,
                   uint8_t *accept_out, int32_t batch, cstr_workspace_t *ws, void *cuda_stream);

/*
 * cstr_step that leaves the input states untouched and writes the new ones to
 * states_out, so that a caller can keep the state after every drafted token
 * (Section 4, Speculative decoding: the target model may reject drafted
 * tokens, so the constraint has to be able to go back to an earlier state).
 *   states_in   DEVICE int32 [batch]
 *   states_out  DEVICE int32 [batch]; may equal states_in (then it is cstr_step)
 * Everything else as in cstr_step.  The same call, over batch x (k + 1) rows
 * whose states are the draft's history q_0 .. q_k of each sequence, penalises
 * the target model's logits at all drafted positions at once with the masks
 * the draft used (the penalties are computed once and serve both models) and decodes
 * the target's own token and next state at each position.
 */
int cstr_step_history(const cstr_table_t *const *tables, int32_t n_tables,
                      const int32_t *row_table, const void *logits, int32_t dtype, int64_t ld,
                      const float *noise, const int32_t *states_in, int32_t *states_out,
                      int32_t *tokens_out, void *masked_out, uint8_t *accept_out, int32_t batch,
                      cstr_workspace_t *ws, void *cuda_stream);

/*
 * Greedy verification and rewind for speculative decoding (Section 4): keep
 * the drafted tokens up to the first position where the target model's token
 * differs, take the target's token there, and rewind the constraint to the
 * state that follows it.
 *   draft_tokens   DEVICE int32 [batch][k]      tokens of the approximation model
 *   target_tokens  DEVICE int32 [batch][k + 1]  target's token at each drafted position
 *                  (and one past the last), from cstr_step_history
 *   target_states  DEVICE int32 [batch][k + 1]  target's next state at each position
 *   n_accepted     DEVICE int32 [batch]         n = drafted tokens kept (0..k)
 *   out_tokens     DEVICE int32 [batch][k + 1]  target_tokens[0..n], then -1
 *   states         DEVICE int32 [batch]         target_states[n]: the rewound state
 * The emitted sequence equals what constrained greedy decoding with the
 * target model alone would produce.  Only enqueues one small kernel.
 */
int cstr_accept_draft(const int32_t *draft_tokens, const int32_t *target_tokens,
                      const int32_t *target_states, int32_t k, int32_t batch,
                      int32_t *n_accepted, int32_t *out_tokens, int32_t *states,
                      void *cuda_stream);

/*
 * Rows since the last call whose input state or table index was out of range
 * (not counting -1), and active rows that had no selectable token.
 * Synchronises cuda_stream, then resets both counters.  Either pointer may be NULL.
 */
int cstr_step_status(cstr_workspace_t *ws, void *cuda_stream, int64_t *bad_state_rows,
                     int64_t *empty_mask_rows);

/* ------------------------------------------------- push-down constraints */

/*
 * Load a deterministic byte-level push-down automaton (Section 3.1: a PDA
 * (Sigma, Pi, S, Q, I, F, E) whose edges are tuples (source, input, pops,
 * target, pushes); before an edge the stack must end with its pops, which it
 * removes, then it appends its pushes).  Sigma is the 256 byte values, Pi the
 * symbols 0 .. n_symbols-1; stacks are written bottom first (last = top).
 *   edge_src, edge_byte, edge_tgt   HOST int32 [n_edges]
 *   pop_off, push_off               HOST int32 [n_edges + 1], non-decreasing from 0
 *   pops, pushes                    HOST int32: edge j pops pops[pop_off[j] .. pop_off[j+1])
 *                                   (last entry = top) and appends pushes[push_off[j] ..
 *                                   push_off[j+1]) in that order
 *   accept                          HOST uint8 [n_states]; acceptance is by final state
 * Limits (CSTR_ERR_PDA otherwise): every edge reads one byte (no epsilon
 * input), pops at most one symbol and pushes at most CSTR_PDA_MAX_PUSH;
 * n_symbols <= CSTR_PDA_MAX_SYMBOLS; the automaton is deterministic: for one
 * (source, byte) either a single edge that pops nothing, or edges that pop
 * pairwise different symbols (the paper's system likewise rejects
 * non-deterministic grammars).  An edge that pops X and pushes X ... reads the
 * top without removing it.  Synchronous; allocates device memory.
 */
#define CSTR_PDA_MAX_PUSH 3
#define CSTR_PDA_MAX_SYMBOLS 254
int cstr_load_pda(const int32_t *edge_src, const int32_t *edge_byte, const int32_t *edge_tgt,
                  const int32_t *pop_off, const int32_t *pops, const int32_t *push_off,
                  const int32_t *pushes, int32_t n_edges, const uint8_t *accept, int32_t n_states,
                  int32_t n_symbols, int32_t start_state, cstr_pda_t **out);
void cstr_free_pda(cstr_pda_t *pda);

/*
 * Build the token-level PDA P_{G o V} = P_G o T_V of Algorithm 3 (Section 3.2;
 * Theorem 3: it accepts a token sequence iff the byte PDA accepts its
 * detokenization).  An edge of P_{G o V} reads a token by chaining the byte
 * edges of its characters, so it may pop and push several symbols.  Stored
 * densely per situation (state q, top-of-stack symbol X or "empty stack"):
 *     mask[q][X] bit v = token v has an edge from q that needs no more of the
 *                        stack than its top symbol X
 *     deep[q][X] bit v = whether v has an edge depends on symbols below X
 *                        (cstr_pda_step decides those against the row's stack)
 * If eos_id >= 0 that token is allowed exactly in accepting states.
 * `pda` and `vocab` must outlive the table.  Limits (CSTR_ERR_SHAPE): at most
 * 65,535 situations (states x (symbols + 1)); no token longer than
 * 255 / (largest push of an edge) bytes.  Device memory: two rows of
 * ceil(V / 32) words per situation and per state.
 * Allocates the table; the build kernel is enqueued on cuda_stream.
 */
int cstr_build_pda_table(const cstr_pda_t *pda, const cstr_vocab_t *vocab, int32_t eos_id,
                         void *cuda_stream, cstr_pda_table_t **out);
void cstr_free_pda_table(cstr_pda_table_t *table);

/*
 * Build the same token-level PDA again into the table's existing storage, with
 * a (possibly different) end-of-sequence token: the compile step of Algorithm 3
 * without any allocation or host synchronisation, only kernels enqueued on
 * cuda_stream.  The table must not be in use by a cstr_pda_step that has not
 * completed.
 */
int cstr_pda_table_rebuild(cstr_pda_table_t *table, int32_t eos_id, void *cuda_stream);

/* Shape of a token-level PDA (any pointer may be NULL). */
int cstr_pda_table_info(const cstr_pda_table_t *table, int32_t *n_states, int32_t *n_symbols,
                        int32_t *vocab_size, int32_t *mask_words, int32_t *start_state);

/*
 * Copy one situation's rows to the host: state in [0, n_states), top a symbol
 * or -1 for the empty stack.
 *   mask_host, deep_host   HOST uint32 [W] or NULL
 * Synchronises cuda_stream first.
 */
int cstr_pda_table_download(const cstr_pda_table_t *table, int32_t state, int32_t top,
                            uint32_t *mask_host, uint32_t *deep_host, void *cuda_stream);

/*
 * Scratch for cstr_pda_step: the step's per-row cells plus one mask row per
 * batch row (for rows whose allowed set depends on more than the top of their
 * stack).  One workspace per stream.
 */
int cstr_pda_workspace_create(const cstr_pda_table_t *table, int32_t max_batch,
                              cstr_pda_workspace_t **out);
void cstr_free_pda_workspace(cstr_pda_workspace_t *ws);

/*
 * One decoding step of Algorithm 3 for `batch` independent rows:
 *   A      = tokens with an edge of P_{G o V} that leaves the row's state q and
 *            whose pops the row's stack s ends with
 *   masked, token: as in cstr_step
 *   the matching edge is traversed: q = its target, its pops leave s, its
 *            pushes are appended
 *   states  DEVICE int32 [batch], in/out (start: the PDA's start state)
 *   stacks  DEVICE int32 [batch][stack_cap], in/out, bottom first
 *   depths  DEVICE int32 [batch], in/out (Algorithm 3 starts from depth 0)
 * logits, dtype, ld, noise, tokens_out, masked_out, accept_out: as in cstr_step.
 * A row whose state is -1 or out of range, whose depth is outside
 * [0, stack_cap] or whose stack holds a symbol outside [0, n_symbols) is
 * inactive: token -1, state -1, all -infinity.  If the traversed edge would
 * leave more than stack_cap symbols the token is still emitted and the row
 * finishes (state -1).  Whenever the new state is -1 the row's stack and depth
 * are left as they were.  Enqueues two kernels on cuda_stream; no
 * allocation, no host synchronisation.
 */
int cstr_pda_step(const cstr_pda_table_t *table, const void *logits, int32_t dtype, int64_t ld,
                  const float *noise, int32_t *states, int32_t *stacks, int32_t *depths,
                  int32_t stack_cap, int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                  int32_t batch, cstr_pda_workspace_t *ws, void *cuda_stream);

/*
 * cstr_pda_step that leaves the rows' situations untouched and writes the new
 * ones to separate arrays, so that a caller can keep the situation after every
 * drafted token (Section 4, Speculative decoding: the constraint has to be able
 * to go back to the situation that followed an earlier token - for a push-down
 * constraint that is the state together with the stack).
 *   states_in, stacks_in, depths_in     DEVICE, read only
 *   states_out, stacks_out, depths_out  DEVICE, same shapes; either all three
 *                                       equal to the inputs (then it is
 *                                       cstr_pda_step) or all three different
 * A row that finishes (new state -1) gets a copy of its old stack and depth.
 * Everything else as in cstr_pda_step.  Over batch x (k + 1) rows holding the
 * draft's history, one call penalises the target model's logits at all drafted
 * positions and decodes the target's own token and next situation at each.
 */
int cstr_pda_step_history(const cstr_pda_table_t *table, const void *logits, int32_t dtype,
                          int64_t ld, const float *noise, const int32_t *states_in,
                          const int32_t *stacks_in, const int32_t *depths_in, int32_t *states_out,
                          int32_t *stacks_out, int32_t *depths_out, int32_t stack_cap,
                          int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                          int32_t batch, cstr_pda_workspace_t *ws, void *cuda_stream);

/*
 * Greedy verification and rewind for speculative decoding under a push-down
 * constraint (Section 4): as cstr_accept_draft, and the rewound situation
 * includes the stack.
 *   draft_tokens   DEVICE int32 [batch][k]
 *   target_tokens, target_states, target_depths   DEVICE int32 [batch][k + 1]
 *   target_stacks  DEVICE int32 [batch][k + 1][stack_cap]
 *   n_accepted     DEVICE int32 [batch]          n = drafted tokens kept
 *   out_tokens     DEVICE int32 [batch][k + 1]   target_tokens[0..n], then -1
 *   states, depths DEVICE int32 [batch];  stacks DEVICE int32 [batch][stack_cap]:
 *                  the target's situation after its token at position n
 * Only enqueues one small kernel.
 */
int cstr_pda_accept_draft(const int32_t *draft_tokens, const int32_t *target_tokens,
                          const int32_t *target_states, const int32_t *target_stacks,
                          const int32_t *target_depths, int32_t k, int32_t batch,
                          int32_t stack_cap, int32_t *n_accepted, int32_t *out_tokens,
                          int32_t *states, int32_t *stacks, int32_t *depths, void *cuda_stream);

/*
 * Rows since the last call that were inactive for another reason than state
 * -1, active rows without a selectable token, and rows that finished because
 * their stack outgrew stack_cap.  Synchronises cuda_stream, then resets the
 * counters.  Any pointer may be NULL.
 */
int cstr_pda_step_status(cstr_pda_workspace_t *ws, void *cuda_stream, int64_t *bad_rows,
                         int64_t *empty_mask_rows, int64_t *overflow_rows);

/*
 * cstr_step without any allocation, for callers that cannot create a
 * workspace.  (The paper has no counterpart; this is a deployment aid.)
 *
 * Some hosts of this library may not call the CUDA allocator once they are
 * running: an inference server that hands all free device memory to its
 * KV-cache pool at start-up, so that a later cudaMalloc can fail; a plug-in
 * that must live inside a memory budget fixed by its host process; a
 * latency-critical decode loop that cannot afford cudaMalloc's device-wide
 * synchronisation.  For them the per-row scratch of the step is a fixed array
 * inside the library image: about 48 KB of device memory on every GPU that
 * loads libcstr, held until the process exits, enough for
 * CSTR_STATIC_MAX_BATCH rows.
 *
 * Arguments, semantics and results are exactly those of cstr_step, without the
 * workspace.  The call allocates nothing (no cudaMalloc / cudaFree, no
 * allocating library routine); it enqueues one small memset and the step
 * kernel on cuda_stream.  batch > CSTR_STATIC_MAX_BATCH is rejected with
 * CSTR_ERR_SHAPE.  The status counters of cstr_step_status are not available
 * here; a row's token of -1 carries the same information.
 *
 * The first call on each device looks up the array's device address (with
 * that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps the previous call's
 * contents, so each call clears it first; two calls that may overlap on the
 * GPU (different streams without an ordering between them) race on it - order
 * them, or use cstr_step with one workspace per stream.
 */
#define CSTR_STATIC_MAX_BATCH 4096
int cstr_step_static(const cstr_table_t *const *tables, int32_t n_tables,
                     const int32_t *row_table, const void *logits, int32_t dtype, int64_t ld,
                     const float *noise, int32_t *states, int32_t *tokens_out, void *masked_out,
                     uint8_t *accept_out, int32_t batch, void *cuda_stream);

/* Message for the calling thread's most recent error ("" if none). */
const char *cstr_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CSTR_H */
