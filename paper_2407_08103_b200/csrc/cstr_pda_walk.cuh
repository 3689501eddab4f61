// Walking a token's bytes through the byte-level PDA (shared by the table
// builder, the per-row resolution of stack-dependent tokens and the step
// kernel's edge traversal).
#pragma once

#include "cstr_internal.cuh"

namespace cstr_pda_dev {

constexpr int kLocMax = 256;   // symbols one token may leave on top of the stack it found

enum { WALK_DEAD = 0, WALK_OK = 1, WALK_DEEP = 2 };

// Chain the byte edges of bytes[0..len) from state q.  The stack found is
// ctx[0..cd) when ctx is non-null (all of it known), else the single symbol
// known_top (cd = 1) or nothing (cd = 0) with `unknown_below` saying whether
// unseen symbols lie underneath.  loc receives what the chain leaves on top.
// WALK_DEEP: the chain reached a byte whose edge depends on an unseen symbol.
__device__ __forceinline__ int pda_walk(const cstr_pda_view &P, int q, const int32_t *ctx, int known_top,
                                        int cd, bool unknown_below, const uint8_t *bytes, int len,
                                        uint8_t *loc, int &q_out, int &cd_out, int &nloc_out)
{
    int nloc = 0;
    if (len <= 0)
        return WALK_DEAD;                           // an empty token never has an edge
    for (int k = 0; k < len; ++k) {
        int t;
        if (nloc > 0) {
            t = loc[nloc - 1];
        } else if (cd > 0) {
            t = ctx ? ctx[cd - 1] : known_top;
            if ((unsigned)t >= (unsigned)P.n_symbols)
                return WALK_DEAD;
        } else {
            t = unknown_below ? P.n_symbols + 1 : P.n_symbols;
        }
        const long long at = ((long long)q * P.NT + t) * 256 + bytes[k];
        if (!CSTR_INB(P.oob, at, P.act_len, CSTR_SITE_PDA))
            return WALK_DEAD;
        const uint32_t a = __ldg(P.act + at);
        if (a == CSTR_PDA_NONE)
            return WALK_DEAD;
        if (a == CSTR_PDA_NEEDCTX)
            return WALK_DEEP;
        if (!CSTR_INB(P.oob, a, P.n_edges, CSTR_SITE_PDA))
            return WALK_DEAD;
        const int2 e = __ldg(P.edge + a);
        const unsigned meta = (unsigned)e.y;
        if (meta >> 28) {                           // pops the symbol it looked at
            if (nloc > 0)
                --nloc;
            else
                --cd;
        }
        const int npush = (meta >> 24) & 7;
        if (nloc + npush > kLocMax)
            return WALK_DEAD;                       // excluded by the build's length check
        for (int i = 0; i < npush; ++i)
            loc[nloc++] = (uint8_t)(meta >> (8 * i));
        q = e.x;
    }
    q_out = q;
    cd_out = cd;
    nloc_out = nloc;
    return WALK_OK;
}

// Traverse the edge of token `tok` for row r (Algorithm 3, edge traversal): walk the
// token's bytes from the row's state and stack, which yields the edge's target
// and stack edit.  `active` = the row had a usable state and stack.
__device__ __forceinline__ void pda_traverse(const cstr_pda_advance &a, int r, bool active, int tok)
{
    const int q = a.states_in[r];
    const int d = a.depths_in[r];
    const int32_t *s_in = a.stacks_in + (long long)r * a.cap;
    int32_t *s_out = a.stacks + (long long)r * a.cap;
    const bool in_place = s_in == s_out;
    int q2 = CSTR_DEAD;
    int keep = (d >= 0 && d <= a.cap) ? d : 0;     // symbols of the old stack that stay
    int d2 = d;
    uint8_t loc[kLocMax];
    int nloc = 0;
    if (!active) {
        if (q != -1)
            atomicAdd(a.counters + 0, 1ull);
    } else if (tok < 0) {
        atomicAdd(a.counters + 1, 1ull);
    } else if (tok != a.eos_id) {
        int qn, cd, nl;
        const uint32_t b0 = a.voff[tok], b1 = a.voff[tok + 1];
        if (pda_walk(a.P, q, s_in, 0, d, false, a.vbytes + b0, (int)(b1 - b0), loc, qn, cd, nl) ==
            WALK_OK) {
            if (cd + nl > a.cap) {
                atomicAdd(a.counters + 2, 1ull);
            } else {
                keep = cd;
                nloc = nl;
                d2 = cd + nl;
                q2 = qn;
            }
        }
    }
    if (!in_place)                                  // the history keeps the old row untouched
        for (int i = 0; i < keep; ++i)
            s_out[i] = s_in[i];
    for (int i = 0; i < nloc; ++i)
        s_out[keep + i] = loc[i];
    a.depths[r] = d2;
    a.states[r] = q2;
    if (a.accept_out)
        a.accept_out[r] = (q2 >= 0) ? (uint8_t)(a.accept[q2] != 0) : (uint8_t)0;
}

}  // namespace cstr_pda_dev
