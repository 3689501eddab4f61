/*
 * ORACLE (test infrastructure, not product code).
 *
 * Plain CPU statement of the push-down variant of the method (Section 3):
 *
 *   - Section 3.1: a PDA (Sigma, Pi, S, Q, I, F, E) has edges
 *     (source, input, pops, target, pushes) with pops, pushes in Pi*.  A word is
 *     accepted if a chain of edges spells it, starts in I, ends in F, and the
 *     stack edits are coherent: before every edge the stack must END WITH the
 *     edge's pops; the edge removes them and appends its pushes.
 *   - Section 3.2: composing the PDA with the detokenizing transducer T_V gives
 *     a PDA over tokens, P_{G o V}(x) = P_G(T_V(x)) (Theorem 3): an edge of
 *     P_{G o V} that reads token v from state q is a chain of byte edges that
 *     spells d(v); its pops are the symbols the chain takes from the stack it
 *     found (in stack order), its pushes what the chain leaves on top.  Edges
 *     may cross terminal boundaries and pop or push several symbols (Figure 7).
 *   - Algorithm 3, loop body: A = inputs of the edges of P_{G o V} that leave q
 *     and whose pops the current stack s ends with; logits outside A become
 *     -infinity; a token is selected; the matching edge e is traversed:
 *     q <- target(e), s <- s[1 : |s| - |pops(e)|] pushes(e).
 *
 * Stacks are written bottom first: s[depth - 1] is the top; "pops" of an edge
 * are listed in the same order (last entry = top of the stack), pushes in the
 * order they are appended.
 *
 * Readings the paper leaves open (kept identical in the library under test):
 *   - the byte PDA is real-time: every edge reads exactly one byte (the paper
 *     allows epsilon inputs; a grammar front-end removes them);
 *   - acceptance is by final state alone (Section 3.1 asks only target in F);
 *   - Algorithm 3 starts from the empty stack; callers may start anywhere;
 *   - a token of zero length never has an edge; the optional end-of-sequence
 *     token is allowed exactly in accepting states and finishes the row;
 *   - selection, ties, NaN, inactive rows: as in the finite-state step;
 *   - stacks live in arrays of `cap` symbols per row.  A row whose state is -1
 *     or out of range, whose depth is outside [0, cap], or whose stack holds a
 *     symbol outside [0, n_symbols) is inactive: token -1, state -1, all
 *     -infinity, stack untouched.  If the traversed edge would leave more than
 *     `cap` symbols, the token is still emitted but the row finishes (state
 *     -1, stack untouched) and counters[2] is bumped.  Whenever the new state
 *     is -1 the stack and depth are left as they were;
 *   - if several edges match (a non-deterministic PDA), the first one in the
 *     caller's edge order of the first differing byte edge wins; the library
 *     under test rejects such automata, so parity never depends on this.
 *
 * No blocking, no tables, nothing shared with the CUDA side.  Built with
 * gcc -O2 -fopenmp -ffp-contract=off.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define DEAD (-1)
#define MAX_CTX 80     /* symbols one token edge may take from the stack it found */
#define MAX_LOC 400    /* symbols one token edge may leave on top                   */

typedef struct {
    int32_t n_states, n_symbols, n_edges;
    const int32_t *src, *inp, *tgt;
    const int32_t *pop_off, *pops, *push_off, *pushes;
    const uint8_t *accept;
    /* edges grouped by (source, input byte), caller's order kept inside a group:
       by[by_off[source * 256 + byte] .. by_off[source * 256 + byte + 1]) */
    int32_t *by_off, *by;
} pda_view;

/* One edge of the token-level PDA P_{G o V} (source and input are implied). */
typedef struct {
    int32_t tgt;
    int32_t npop;
    int32_t pops[MAX_CTX];    /* stack order: pops[npop - 1] was the top */
    int32_t npush;
    int32_t pushes[MAX_LOC];
} tok_edge;

typedef struct {
    tok_edge *out;
    int32_t n, cap;
    int32_t overflow;         /* a bound above was hit (reported, never silent) */
} edge_sink;

/*
 * Chains of byte edges that spell bytes[k..end) from state cur.  ctx holds the
 * symbols taken so far from the stack the chain found (ctx[0] = its top, taken
 * first), loc what the chain has pushed and not yet popped again.
 */
static void compose(const pda_view *P, int32_t cur, const uint8_t *bytes, int64_t k, int64_t end,
                    const int32_t *ctx, int32_t nctx, const int32_t *loc, int32_t nloc,
                    edge_sink *sink)
{
    if (k == end) {
        if (sink->n >= sink->cap) {
            sink->overflow = 1;
            return;
        }
        tok_edge *e = &sink->out[sink->n++];
        e->tgt = cur;
        e->npop = nctx;
        for (int32_t i = 0; i < nctx; ++i)
            e->pops[i] = ctx[nctx - 1 - i];      /* deepest symbol first */
        e->npush = nloc;
        memcpy(e->pushes, loc, (size_t)nloc * sizeof(int32_t));
        return;
    }
    const int64_t g = (int64_t)cur * 256 + bytes[k];
    for (int32_t jj = P->by_off[g]; jj < P->by_off[g + 1]; ++jj) {
        const int32_t j = P->by[jj];
        int32_t ctx2[MAX_CTX], loc2[MAX_LOC];
        int32_t nctx2 = nctx, nloc2 = nloc, ok = 1;
        memcpy(ctx2, ctx, (size_t)nctx * sizeof(int32_t));
        memcpy(loc2, loc, (size_t)nloc * sizeof(int32_t));
        /* the stack must end with the edge's pops: match them top first */
        for (int32_t i = P->pop_off[j + 1] - 1; i >= P->pop_off[j] && ok; --i) {
            const int32_t sym = P->pops[i];
            if (nloc2 > 0) {
                if (loc2[nloc2 - 1] != sym)
                    ok = 0;                       /* incoherent stack edits */
                else
                    nloc2 -= 1;
            } else if (nctx2 < MAX_CTX) {
                ctx2[nctx2++] = sym;              /* a demand on the stack found */
            } else {
                sink->overflow = 1;
                ok = 0;
            }
        }
        if (!ok)
            continue;
        for (int32_t i = P->push_off[j]; i < P->push_off[j + 1]; ++i) {
            if (nloc2 >= MAX_LOC) {
                sink->overflow = 1;
                ok = 0;
                break;
            }
            loc2[nloc2++] = P->pushes[i];
        }
        if (ok)
            compose(P, P->tgt[j], bytes, k + 1, end, ctx2, nctx2, loc2, nloc2, sink);
    }
}

/* Edges of P_{G o V} with source q and input token v (an empty token has none). */
static int32_t token_edges(const pda_view *P, int32_t q, const uint8_t *bytes, int64_t begin,
                           int64_t end, tok_edge *out, int32_t cap, int32_t *overflow)
{
    edge_sink sink = {out, 0, cap, 0};
    if (end > begin)
        compose(P, q, bytes, begin, end, 0, 0, 0, 0, &sink);
    if (overflow && sink.overflow)
        *overflow = 1;
    return sink.n;
}

/* "s ends with pops(e)" */
static int ends_with(const int32_t *s, int32_t depth, const tok_edge *e)
{
    if (e->npop > depth)
        return 0;
    for (int32_t i = 0; i < e->npop; ++i)
        if (s[depth - e->npop + i] != e->pops[i])
            return 0;
    return 1;
}

#define EDGE_CAP 512

/* The edge Algorithm 3 traverses for token v from (q, s), or NULL if v is not in A. */
static const tok_edge *matching_edge(const pda_view *P, int32_t q, const int32_t *s, int32_t depth,
                                     const uint8_t *bytes, const int64_t *off, int32_t v,
                                     tok_edge *buf, int32_t *overflow)
{
    const int32_t n = token_edges(P, q, bytes, off[v], off[v + 1], buf, EDGE_CAP, overflow);
    for (int32_t i = 0; i < n; ++i)
        if (ends_with(s, depth, &buf[i]))
            return &buf[i];
    return 0;
}

/* ------------------------------------------------------------------ exported */

static pda_view make_view(int32_t n_states, int32_t n_symbols, int32_t n_edges, const int32_t *src,
                          const int32_t *inp, const int32_t *tgt, const int32_t *pop_off,
                          const int32_t *pops, const int32_t *push_off, const int32_t *pushes,
                          const uint8_t *accept)
{
    pda_view P = {n_states, n_symbols, n_edges, src, inp, tgt, pop_off, pops, push_off, pushes,
                  accept, 0, 0};
    const int64_t groups = (int64_t)n_states * 256;
    P.by_off = (int32_t *)calloc((size_t)groups + 1, sizeof(int32_t));
    P.by = (int32_t *)malloc(((size_t)n_edges + 1) * sizeof(int32_t));
    for (int32_t j = 0; j < n_edges; ++j)
        P.by_off[(int64_t)src[j] * 256 + inp[j] + 1] += 1;
    for (int64_t g = 0; g < groups; ++g)
        P.by_off[g + 1] += P.by_off[g];
    int32_t *fill = (int32_t *)malloc((size_t)groups * sizeof(int32_t));
    memcpy(fill, P.by_off, (size_t)groups * sizeof(int32_t));
    for (int32_t j = 0; j < n_edges; ++j)
        P.by[fill[(int64_t)src[j] * 256 + inp[j]]++] = j;
    free(fill);
    return P;
}

static void free_view(pda_view *P)
{
    free(P->by_off);
    free(P->by);
}

/*
 * Section 3.1 acceptance, by the definition: is there a chain of edges that
 * spells w, starts at `start` with stack init[0..n_init) and ends in F?
 * Depth-first over all edges (non-deterministic automata included).
 */
static int accepts_from(const pda_view *P, int32_t q, int32_t *s, int32_t depth, int32_t cap,
                        const uint8_t *w, int64_t k, int64_t n)
{
    if (k == n)
        return P->accept[q] != 0;
    const int64_t g = (int64_t)q * 256 + w[k];
    for (int32_t jj = P->by_off[g]; jj < P->by_off[g + 1]; ++jj) {
        const int32_t j = P->by[jj];
        const int32_t np = P->pop_off[j + 1] - P->pop_off[j];
        const int32_t nu = P->push_off[j + 1] - P->push_off[j];
        if (np > depth || depth - np + nu > cap)
            continue;
        if (memcmp(s + depth - np, P->pops + P->pop_off[j], (size_t)np * sizeof(int32_t)) != 0)
            continue;
        int32_t saved[MAX_CTX];
        if (np > MAX_CTX)
            continue;
        memcpy(saved, s + depth - np, (size_t)np * sizeof(int32_t));
        memcpy(s + depth - np, P->pushes + P->push_off[j], (size_t)nu * sizeof(int32_t));
        const int hit = accepts_from(P, P->tgt[j], s, depth - np + nu, cap, w, k + 1, n);
        memcpy(s + depth - np, saved, (size_t)np * sizeof(int32_t));   /* undo */
        if (hit)
            return 1;
    }
    return 0;
}

/* accepted[i] = 1 iff the PDA accepts words[woff[i] .. woff[i+1]). */
void oracle_pda_accepts(int32_t n_states, int32_t n_symbols, int32_t n_edges, const int32_t *src,
                        const int32_t *inp, const int32_t *tgt, const int32_t *pop_off,
                        const int32_t *pops, const int32_t *push_off, const int32_t *pushes,
                        const uint8_t *accept, int32_t start, const int32_t *init, int32_t n_init,
                        const uint8_t *words, const int64_t *woff, int64_t n_words,
                        uint8_t *accepted, int32_t threads)
{
    pda_view P = make_view(n_states, n_symbols, n_edges, src, inp, tgt, pop_off, pops,
                                 push_off, pushes, accept);
#pragma omp parallel for num_threads(threads) schedule(dynamic, 64)
    for (int64_t i = 0; i < n_words; ++i) {
        const int64_t len = woff[i + 1] - woff[i];
        const int32_t cap = n_init + (int32_t)len * 8 + 8;
        int32_t *s = (int32_t *)malloc((size_t)cap * sizeof(int32_t));
        memcpy(s, init, (size_t)n_init * sizeof(int32_t));
        accepted[i] = (uint8_t)accepts_from(&P, start, s, n_init, cap, words + woff[i], 0, len);
        free(s);
    }
    free_view(&P);
}

/*
 * Edges of P_{G o V} leaving state q on token bytes[0..len): up to max_edges
 * records of `stride` int32 each: [target, npop, npush, pops..., pushes...].
 * Returns the number of edges, or -1 if a bound was exceeded.
 */
int32_t oracle_pda_token_edges(int32_t n_states, int32_t n_symbols, int32_t n_edges,
                               const int32_t *src, const int32_t *inp, const int32_t *tgt,
                               const int32_t *pop_off, const int32_t *pops,
                               const int32_t *push_off, const int32_t *pushes,
                               const uint8_t *accept, int32_t q, const uint8_t *bytes, int64_t len,
                               int32_t *out, int32_t stride, int32_t max_edges)
{
    pda_view P = make_view(n_states, n_symbols, n_edges, src, inp, tgt, pop_off, pops,
                                 push_off, pushes, accept);
    tok_edge *buf = (tok_edge *)malloc((size_t)max_edges * sizeof(tok_edge));
    int32_t overflow = 0;
    const int32_t n = token_edges(&P, q, bytes, 0, len, buf, max_edges, &overflow);
    for (int32_t i = 0; i < n && !overflow; ++i) {
        int32_t *rec = out + (int64_t)i * stride;
        if (3 + buf[i].npop + buf[i].npush > stride) {
            overflow = 1;
            break;
        }
        rec[0] = buf[i].tgt;
        rec[1] = buf[i].npop;
        rec[2] = buf[i].npush;
        memcpy(rec + 3, buf[i].pops, (size_t)buf[i].npop * sizeof(int32_t));
        memcpy(rec + 3 + buf[i].npop, buf[i].pushes, (size_t)buf[i].npush * sizeof(int32_t));
    }
    free(buf);
    free_view(&P);
    return overflow ? -1 : n;
}

/*
 * Allowed sets for n_cfg situations (q[i], stack stacks[i*cap .. +depth[i])):
 * mask_out[i*W + v/32] bit v%32 = 1 iff token v is in A of Algorithm 3.
 * The end-of-sequence token (if any) is in A iff q is accepting.
 * Returns 1 if an internal bound was exceeded (the result is then not to be used).
 */
int32_t oracle_pda_allowed(int32_t n_states, int32_t n_symbols, int32_t n_edges, const int32_t *src,
                        const int32_t *inp, const int32_t *tgt, const int32_t *pop_off,
                        const int32_t *pops, const int32_t *push_off, const int32_t *pushes,
                        const uint8_t *accept, const uint8_t *bytes, const int64_t *off, int32_t V,
                        int32_t eos_id, const int32_t *q, const int32_t *stacks,
                        const int32_t *depth, int32_t cap, int32_t n_cfg, uint32_t *mask_out,
                        int32_t threads)
{
    pda_view P = make_view(n_states, n_symbols, n_edges, src, inp, tgt, pop_off, pops,
                                 push_off, pushes, accept);
    const int64_t W = ((int64_t)V + 31) / 32;
    int32_t overflow = 0;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1) reduction(| : overflow)
    for (int32_t i = 0; i < n_cfg; ++i) {
        tok_edge *buf = (tok_edge *)malloc(EDGE_CAP * sizeof(tok_edge));
        uint32_t *row = mask_out + (int64_t)i * W;
        memset(row, 0, (size_t)W * sizeof(uint32_t));
        for (int32_t v = 0; v < V; ++v) {
            int ok;
            if (v == eos_id)
                ok = accept[q[i]] != 0;
            else
                ok = matching_edge(&P, q[i], stacks + (int64_t)i * cap, depth[i], bytes, off, v,
                                   buf, &overflow) != 0;
            if (ok)
                row[v >> 5] |= (uint32_t)1 << (v & 31);
        }
        free(buf);
    }
    free_view(&P);
    return overflow;
}

static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/*
 * One constrained decoding step of Algorithm 3 for `batch` rows.
 * states [batch], stacks [batch][cap], depth [batch]: in/out.
 * counters[0] += inactive rows other than state -1; counters[1] += active rows
 * without a selectable token; counters[2] += rows whose stack outgrew cap;
 * counters[3] is set non-zero if an internal bound was exceeded.
 */
void oracle_pda_step(int32_t n_states, int32_t n_symbols, int32_t n_edges, const int32_t *src,
                     const int32_t *inp, const int32_t *tgt, const int32_t *pop_off,
                     const int32_t *pops, const int32_t *push_off, const int32_t *pushes,
                     const uint8_t *accept, const uint8_t *bytes, const int64_t *off, int32_t V,
                     int32_t eos_id, const void *logits, int32_t dtype, int64_t ld,
                     const float *noise, int32_t *states, int32_t *stacks, int32_t *depth,
                     int32_t cap, int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                     int32_t batch, int64_t *counters, int32_t threads)
{
    pda_view P = make_view(n_states, n_symbols, n_edges, src, inp, tgt, pop_off, pops,
                                 push_off, pushes, accept);
    int64_t bad = 0, empty = 0, over = 0;
    int32_t overflow = 0;
#pragma omp parallel for num_threads(threads) schedule(dynamic, 1) reduction(+ : bad, empty, over) \
    reduction(| : overflow)
    for (int32_t r = 0; r < batch; ++r) {
        tok_edge *buf = (tok_edge *)malloc(EDGE_CAP * sizeof(tok_edge));
        const int32_t q = states[r];
        int32_t *s = stacks + (int64_t)r * cap;
        const int32_t d = depth[r];
        const float *lf = (const float *)logits + (int64_t)r * ld;
        const uint16_t *lh = (const uint16_t *)logits + (int64_t)r * ld;
        float *of = (float *)masked_out + (int64_t)r * ld;
        uint16_t *oh = (uint16_t *)masked_out + (int64_t)r * ld;
        const float *nz = noise ? noise + (int64_t)r * ld : 0;
        int active = q >= 0 && q < n_states && d >= 0 && d <= cap;
        for (int32_t i = 0; active && i < d; ++i)
            if (s[i] < 0 || s[i] >= n_symbols)
                active = 0;
        if (!active && q != -1)
            bad += 1;
        float best = -INFINITY;
        int32_t best_v = -1;
        for (int32_t v = 0; v < V; ++v) {
            int ok = 0;
            if (active)
                ok = (v == eos_id) ? (accept[q] != 0)
                                   : (matching_edge(&P, q, s, d, bytes, off, v, buf, &overflow) != 0);
            if (!ok) {
                if (dtype == 0)
                    of[v] = -INFINITY;
                else
                    oh[v] = 0xFF80;
                continue;
            }
            float x;
            if (dtype == 0) {
                x = lf[v];
                memcpy(&of[v], &lf[v], sizeof(float));
            } else {
                x = bf16_to_float(lh[v]);
                oh[v] = lh[v];
            }
            if (nz)
                x = x + nz[v];
            if (x != x)
                continue;
            if (best_v < 0 || x > best) {
                best = x;
                best_v = v;
            }
        }
        if (active && best_v < 0)
            empty += 1;
        tokens_out[r] = best_v;
        int32_t q2 = DEAD;
        if (best_v >= 0 && best_v != eos_id) {
            const tok_edge *e = matching_edge(&P, q, s, d, bytes, off, best_v, buf, 0);
            const int32_t m = d - e->npop;
            if (m + e->npush > cap) {
                over += 1;
            } else {
                memcpy(s + m, e->pushes, (size_t)e->npush * sizeof(int32_t));
                depth[r] = m + e->npush;
                q2 = e->tgt;
            }
        }
        states[r] = q2;
        if (accept_out)
            accept_out[r] = (q2 >= 0) ? (accept[q2] != 0) : 0;
        free(buf);
    }
    counters[0] += bad;
    counters[1] += empty;
    counters[2] += over;
    counters[3] |= overflow;
    free_view(&P);
}
