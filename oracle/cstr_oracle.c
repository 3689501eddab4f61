/*
 * ORACLE (test infrastructure, not product code).
 *
 * Plain CPU statement of what the token-level automaton and the constrained
 * decoding step compute, written from the paper's definitions:
 *
 *   - Algorithm 1 + FSA/FST composition (Section 2.2, "A' = A2 o T1 ...
 *     A'(w) = A2(T1(w))") + Theorem 2: the detokenizing transducer turns a
 *     token v into its characters d(v), so the edge of the token automaton
 *     labelled v that leaves state q ends in the state the character DFA
 *     reaches from q after reading d(v), and exists iff that walk never
 *     leaves the DFA.
 *   - Algorithm 2, decoding loop: A = tokens on outbound edges of q; logits of
 *     tokens outside A become -infinity; a token is selected; q moves along
 *     its edge.
 *
 *   - Section 2.5.1, terminal labels: a state may also have edges labelled with
 *     terminal labels (symbols outside the byte alphabet), each label standing
 *     for a pre-computed set of tokens.  Such an edge allows every token of the
 *     label's set at once (the whole set is OR-ed into the allowed tokens);
 *     when the selected token has no ordinary edge, the terminal edge of the
 *     first label (a fixed precedence: ascending label index) whose set holds
 *     the token is taken - the paper's heuristic for the ambiguity: ordinary
 *     token edges win, then a fixed order over the labels.
 *
 * Readings the paper leaves open (kept identical in the library under test):
 *   - a token of zero length never has an edge (Algorithm 1 emits the last
 *     character of every token, so it assumes |v| >= 1);
 *   - optional end-of-sequence token: allowed exactly in accepting states,
 *     and taking it finishes the row (state -1);
 *   - selection is greedy: the allowed token with the largest
 *     fp32(logit) (+ fp32 noise when supplied, one rounded fp32 addition);
 *     among equal values the lowest token id; NaN never wins; an allowed
 *     token whose value is -infinity still beats "no token";
 *   - a row whose state is -1 or out of range, or that has no winner, yields
 *     token -1 and state -1, with every masked logit -infinity.
 *
 * No blocking, no tables shared with the CUDA side, no tuning.  Built with
 * gcc -O2 -fopenmp -ffp-contract=off; rows / states are independent, so the
 * outer loops carry a plain "omp parallel for".
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define DEAD (-1)

/* delta*(q, d(v)): walk the bytes of one token from state q. */
static int32_t walk_token(const int32_t *trans, int32_t q, const uint8_t *bytes,
                          int64_t begin, int64_t end)
{
    if (end <= begin)
        return DEAD; /* empty token: no edge */
    int32_t s = q;
    for (int64_t k = begin; k < end; ++k) {
        s = trans[(int64_t)s * 256 + bytes[k]];
        if (s < 0)
            return DEAD;
    }
    return s;
}

/* A DFA with optional terminal-label edges: term[q * n_term + t] = target or -1. */
typedef struct {
    const int32_t *trans;
    const uint8_t *accept;
    const int32_t *term;   /* may be NULL when n_term == 0 */
    int32_t n_term;
} dfa_view;

/* First terminal edge of q, in label order, whose token set holds v (tmask bit). */
static int32_t terminal_edge(const dfa_view *d, int32_t q, const uint32_t *tmask, int32_t v)
{
    if (d->n_term == 0 || !tmask)
        return DEAD;
    for (int32_t t = 0; t < d->n_term; ++t) {
        int32_t target = d->term[(int64_t)q * d->n_term + t];
        if (target >= 0 && ((tmask[v] >> t) & 1u))
            return target;
    }
    return DEAD;
}

/* Edge of the token automaton: target state of token v from state q, or DEAD. */
static int32_t token_edge(const dfa_view *d, int32_t q, const uint8_t *bytes, const int64_t *off,
                          const uint32_t *tmask, int32_t v, int32_t eos_id)
{
    if (v == eos_id)
        return DEAD; /* taking EOS finishes the row; whether it is allowed is separate */
    if (off[v + 1] <= off[v])
        return DEAD; /* empty token: no edge of either kind */
    int32_t s = walk_token(d->trans, q, bytes, off[v], off[v + 1]);
    if (s >= 0)
        return s;    /* ordinary edges come first */
    return terminal_edge(d, q, tmask, v);
}

static int token_allowed(const dfa_view *d, int32_t q, const uint8_t *bytes, const int64_t *off,
                         const uint32_t *tmask, int32_t v, int32_t eos_id)
{
    if (v == eos_id)
        return d->accept[q] != 0;
    return token_edge(d, q, bytes, off, tmask, v, eos_id) >= 0;
}

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Token table for states q_lo <= q < q_hi:
 *   next_out[(q - q_lo) * V + v] = target state or -1
 *   mask_out[(q - q_lo) * W + v / 32] bit (v % 32) = 1 iff token v is allowed in q
 * W = ceil(V / 32); unused high bits of the last word are 0.
 */
void oracle_token_table(const int32_t *trans, const uint8_t *accept, int32_t n_states,
                        const int32_t *term_trans, int32_t n_term, const uint32_t *tmask,
                        const uint8_t *bytes, const int64_t *off, int32_t V, int32_t eos_id,
                        int32_t q_lo, int32_t q_hi, int32_t *next_out, uint32_t *mask_out,
                        int32_t threads)
{
    const int64_t W = ((int64_t)V + 31) / 32;
    const dfa_view d = {trans, accept, term_trans, term_trans ? n_term : 0};
    (void)n_states;
#pragma omp parallel for num_threads(threads) schedule(static)
    for (int32_t q = q_lo; q < q_hi; ++q) {
        int32_t *nrow = next_out + (int64_t)(q - q_lo) * V;
        uint32_t *mrow = mask_out + (int64_t)(q - q_lo) * W;
        memset(mrow, 0, (size_t)W * sizeof(uint32_t));
        for (int32_t v = 0; v < V; ++v) {
            nrow[v] = token_edge(&d, q, bytes, off, tmask, v, eos_id);
            if (token_allowed(&d, q, bytes, off, tmask, v, eos_id))
                mrow[v >> 5] |= (uint32_t)1 << (v & 31);
        }
    }
}

static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * One constrained decoding step for `batch` rows (Algorithm 2, loop body).
 *
 * tables: n_tables DFAs given as arrays of pointers (trans[t], accept[t],
 * n_states[t], and optionally term_trans[t] with n_term[t] labels; tmask[v] has
 * bit t set iff token v belongs to the set of label t); row r uses table
 * row_table[r] (or 0 when row_table is NULL).
 * logits: [batch][ld] fp32 (dtype 0) or bf16 bit patterns (dtype 1);
 * noise: [batch][ld] fp32 or NULL.  masked_out: same shape/dtype as logits,
 * columns >= V are not written.  states: in/out.  counters[0] += rows whose
 * input state was below -1 or >= n_states; counters[1] += active rows with no
 * selectable token.
 */
void oracle_step(const int32_t *const *trans, const uint8_t *const *accept,
                 const int32_t *n_states, const int32_t *const *term_trans,
                 const int32_t *n_term, const uint32_t *tmask, int32_t n_tables,
                 const int32_t *row_table,
                 const uint8_t *bytes, const int64_t *off, int32_t V, int32_t eos_id,
                 const void *logits, int32_t dtype, int64_t ld, const float *noise,
                 int32_t *states, int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                 int32_t batch, int64_t *counters, int32_t threads)
{
    int64_t bad = 0, empty = 0;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1) reduction(+ : bad, empty)
    for (int32_t r = 0; r < batch; ++r) {
        int32_t t = row_table ? row_table[r] : 0;
        int32_t q = states[r];
        const float *lf = (const float *)logits + (int64_t)r * ld;
        const uint16_t *lh = (const uint16_t *)logits + (int64_t)r * ld;
        float *of = (float *)masked_out + (int64_t)r * ld;
        uint16_t *oh = (uint16_t *)masked_out + (int64_t)r * ld;
        const float *nz = noise ? noise + (int64_t)r * ld : 0;
        int active = (t >= 0 && t < n_tables && q >= 0 && q < n_states[t]);
        if (!active && q != -1)
            bad += 1;
        dfa_view d = {0, 0, 0, 0};
        if (active) {
            d.trans = trans[t];
            d.accept = accept[t];
            d.term = term_trans ? term_trans[t] : 0;
            d.n_term = (term_trans && term_trans[t]) ? n_term[t] : 0;
        }
        float best = -INFINITY;
        int32_t best_v = -1;
        for (int32_t v = 0; v < V; ++v) {
            int ok = active && token_allowed(&d, q, bytes, off, tmask, v, eos_id);
            if (!ok) {
                if (dtype == 0)
                    of[v] = -INFINITY;
                else
                    oh[v] = 0xFF80; /* bf16 -infinity */
                continue;
            }
            float x;
            if (dtype == 0) {
                x = lf[v];
                memcpy(&of[v], &lf[v], sizeof(float)); /* untouched: bit copy */
            } else {
                x = bf16_to_float(lh[v]);
                oh[v] = lh[v];
            }
            if (nz)
                x = x + nz[v];
            if (x != x)
                continue; /* NaN never wins */
            if (best_v < 0 || x > best) {
                best = x;
                best_v = v;
            }
        }
        if (active && best_v < 0)
            empty += 1;
        tokens_out[r] = best_v;
        int32_t q2 = DEAD;
        if (best_v >= 0)
            q2 = token_edge(&d, q, bytes, off, tmask, best_v, eos_id);
        states[r] = q2;
        if (accept_out)
            accept_out[r] = (q2 >= 0) ? (accept[t][q2] != 0) : 0;
    }
    counters[0] += bad;
    counters[1] += empty;
}

/*
 * Speculative decoding, greedy verification and rewind (Section 4): the target
 * model accepts a prefix of the drafted tokens; the constraint, which kept the
 * state reached after every drafted token rather than only the latest one,
 * restarts from the state that follows the last token kept.  With greedy selection the kept prefix is the
 * run of positions where the target's own (constrained) token equals the
 * drafted one, and the target's token at the first disagreement (or after the
 * last drafted position) is emitted as well.
 *   draft[b][k], tgt_tok[b][k+1], tgt_state[b][k+1] ->
 *   n_accepted[b], out_tokens[b][k+1] (tgt_tok[0..n], then -1), states[b] = tgt_state[n]
 */
void oracle_accept_draft(const int32_t *draft, const int32_t *tgt_tok, const int32_t *tgt_state,
                         int32_t k, int32_t batch, int32_t *n_accepted, int32_t *out_tokens,
                         int32_t *states)
{
    for (int32_t r = 0; r < batch; ++r) {
        const int32_t *d = draft + (int64_t)r * k;
        const int32_t *t = tgt_tok + (int64_t)r * (k + 1);
        int32_t n = 0;
        while (n < k && d[n] == t[n])
            n += 1;
        for (int32_t i = 0; i <= k; ++i)
            out_tokens[(int64_t)r * (k + 1) + i] = (i <= n) ? t[i] : -1;
        n_accepted[r] = n;
        states[r] = tgt_state[(int64_t)r * (k + 1) + n];
    }
}
