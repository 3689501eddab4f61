// Fused constrained decoding step (Algorithm 2, loop body) for a batch of rows:
// mask from the row's state, -inf on disallowed logits, arg-max selection with
// lowest-index tie-break (optionally over logit + supplied noise), next-state
// update - one streaming pass over the logits, one kernel.
//
// A row is split into chunks of whole tiles; one CTA streams one chunk with
// 128-bit loads/stores, applying the state's bitmask a 32-token word at a time
// (one coalesced word load per lane per tile, words handed around with
// shuffles).  Each CTA folds its (value, index) winner into a per-row 64-bit
// cell with atomicMax on an order-preserving key - a total order, so the
// result does not depend on arrival order - and the CTA that arrives last at
// the row's ticket reads the cell, emits token / state / accept flag and
// resets the scratch.  Nobody waits on anybody.
#include <cuda_bf16.h>
#include <math_constants.h>
#include <string.h>

#include <mutex>

#include "cstr_internal.cuh"
#include "cstr_pda_walk.cuh"

namespace {

struct TableDesc {
    const uint32_t *mask;
    const void *next;
    const uint8_t *accept;
    const int32_t *rank;     // caller's state id -> index into a row of next, or null (identity)
    const int32_t *unrank;   // and back
    long long lds;       // next is token-major: next[token * lds + state]
    long long ldw;
    int n_states;
    int wide;
    int code_shift;
};

struct StepParams {
    TableDesc tab[CSTR_MAX_TABLES];
    const int32_t *row_table;
    const void *logits;
    const float *noise;
    void *out;
    const int32_t *states;   // per-row state before the step
    int32_t *states_out;     // state after the step (may be the same array)
    int32_t *tokens;
    uint8_t *accept_out;
    unsigned long long *cell;
    unsigned int *ticket;
    unsigned long long *counters;
    const uint32_t *const *row_mask;   // push-down kernels: per-row mask pointers, no tables
    cstr_pda_advance pda;              // push-down kernels: what the edge traversal needs
    long long ld;
    int V;
    int n_tables;
    int batch;           // rows; extent of the per-row arrays
    unsigned long long *oob;   // checking build: bounds record (null in the release build)
    int nchunks;         // CTAs per row
    int tiles_per_cta;
    int tile_tokens;     // tokens per warp tile of the launched kernel
};

// 16-byte vectors in flight per lane per tile: 8 for the greedy kernels, 4 when a
// noise stream is read as well (keeps the register count at four CTAs per SM).
__host__ __device__ constexpr int unroll_for(bool noise) { return noise ? 4 : 8; }
constexpr unsigned kFull = 0xffffffffu;

struct Best {
    float v;
    int i;   // -1: nothing selected yet
};

// Scan-order update: indices arrive in increasing order within a thread, so a
// later candidate wins only if strictly larger (or if nothing is held yet).
// `cand` is NaN for disallowed positions, so they never win.
__device__ __forceinline__ void consider(Best &b, float cand, int idx)
{
    const bool take = (cand > b.v) || (b.i < 0 && cand == cand);
    b.v = take ? cand : b.v;
    b.i = take ? idx : b.i;
}

// Order-free merge of two partial winners.
__device__ __forceinline__ void merge(Best &b, float ov, int oi)
{
    const bool take = oi >= 0 && (b.i < 0 || ov > b.v || (ov == b.v && oi < b.i));
    b.v = take ? ov : b.v;
    b.i = take ? oi : b.i;
}

// Monotone map float -> uint32 (after folding -0 into +0), then (key, ~index).
__device__ __forceinline__ unsigned long long pack_key(float v, int idx)
{
    v = v + 0.0f;                                   // -0.0 + 0.0 = +0.0 (round to nearest)
    const unsigned u = __float_as_uint(v);
    const unsigned hi = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)hi << 32) | (unsigned long long)(0xffffffffu - (unsigned)idx);
}

struct RowCtx {
    int r, chunk, t, q;
    bool active;
    const uint32_t *mrow;
};

template <bool PDA>
__device__ __forceinline__ RowCtx row_context(const StepParams &p)
{
    RowCtx c;
    c.r = blockIdx.x / p.nchunks;
    c.chunk = blockIdx.x - c.r * p.nchunks;
    if (!CSTR_INB(p.oob, c.r, p.batch, CSTR_SITE_STEP_ROW)) {   // cannot happen: grid = batch x nchunks
        c.r = 0;
        c.t = 0;
        c.q = -1;
        c.active = false;
        c.mrow = nullptr;
        return c;
    }
    if (PDA) {                                      // the rows' masks were resolved beforehand
        c.t = 0;
        c.q = 0;
        c.mrow = p.row_mask[c.r];
        c.active = c.mrow != nullptr;
        return c;
    }
    c.t = p.row_table ? p.row_table[c.r] : 0;
    c.q = p.states[c.r];
    const bool table_ok = c.t >= 0 && c.t < p.n_tables;
    const int tt = table_ok ? c.t : 0;
    c.active = table_ok && c.q >= 0 && c.q < p.tab[tt].n_states;
    c.t = tt;
    c.mrow = c.active ? p.tab[tt].mask + (long long)c.q * p.tab[tt].ldw : nullptr;
    return c;
}

// CTA-level reduction, cross-CTA fold, and the last arriver's finalisation.
template <bool PDA>
__device__ __forceinline__ void finish_row(const StepParams &p, const RowCtx &c, Best b)
{
    __shared__ float s_v[32];
    __shared__ int s_i[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_down_sync(kFull, b.v, off);
        const int oi = __shfl_down_sync(kFull, b.i, off);
        merge(b, ov, oi);
    }
    if (lane == 0) {
        s_v[warp] = b.v;
        s_i[warp] = b.i;
    }
    __syncthreads();
    if (threadIdx.x != 0)
        return;
    const int nwarps = (blockDim.x + 31) >> 5;
    for (int w = 1; w < nwarps; ++w)
        merge(b, s_v[w], s_i[w]);
    if (b.i >= 0)
        atomicMax(p.cell + c.r, pack_key(b.v, b.i));
    __threadfence();
    const unsigned prev = atomicAdd(p.ticket + c.r, 1u);
    if (prev != (unsigned)p.nchunks - 1u)
        return;
    __threadfence();
    const unsigned long long key = atomicExch(p.cell + c.r, 0ull);
    p.ticket[c.r] = 0u;
    if (PDA) {                                      // Algorithm 3: traverse the token's edge
        const int t = (c.active && key != 0ull)
                          ? (int)(0xffffffffu - (unsigned)(key & 0xffffffffull)) : -1;
        p.tokens[c.r] = t;
        cstr_pda_dev::pda_traverse(p.pda, c.r, c.active, t);
        return;
    }
    int tok = -1, q2 = CSTR_DEAD;
    const TableDesc &tb = p.tab[c.t];
    if (c.active && key != 0ull) {
        tok = (int)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        // next is indexed by, and holds, the builder's internal state ids
        const long long at = (long long)tok * tb.lds + (tb.rank ? tb.rank[c.q] : c.q);
        if (!CSTR_INB(p.oob, at, (long long)p.V * tb.lds, CSTR_SITE_STEP_NEXT) ||
            !CSTR_INB(p.oob, tok, p.V, CSTR_SITE_STEP_NEXT))
            q2 = tb.n_states << tb.code_shift;          // decodes to "no edge"
        else
        q2 = tb.wide ? ((const int32_t *)tb.next)[at] : (int)((const uint16_t *)tb.next)[at];
        q2 = q2 >> tb.code_shift;                       // entries are codes of permuted ids ...
        q2 = CSTR_UNPERM(q2);
        if (q2 == tb.n_states)
            q2 = CSTR_DEAD;                             // ... and the sink n_states means "no edge"
        else if (tb.unrank)
            q2 = tb.unrank[q2];
    } else if (c.active) {
        atomicAdd(p.counters + 1, 1ull);
    } else if (c.q != -1) {
        atomicAdd(p.counters + 0, 1ull);
    }
    p.tokens[c.r] = tok;
    p.states_out[c.r] = q2;
    if (p.accept_out)
        p.accept_out[c.r] = (q2 >= 0 && CSTR_INB(p.oob, q2, tb.n_states, CSTR_SITE_STEP_NEXT))
                                ? (uint8_t)(tb.accept[q2] != 0) : (uint8_t)0;
}

// ---- per-vector processing ------------------------------------------------
//
// The streaming loop tracks the winner at vector granularity only: the largest
// candidate of each 16-byte vector (NaN where nothing in it can win) and the
// first vector that holds the running maximum.  Which element of that vector
// it is gets resolved once per warp after the loop (refine_winner), which
// keeps the per-logit work to two selects and one max.

struct VBest {
    float v;
    int vec;   // token index of the winning vector's first element; -1: none yet
};

__device__ __forceinline__ void vconsider(VBest &b, float m, int tok)
{
    const bool take = (m > b.v) || (b.vec < 0 && m == m);
    b.v = take ? m : b.v;
    b.vec = take ? tok : b.vec;
}

// fp32: 4 logits per 16-byte vector, mask bits in bits[3:0].
template <bool NOISE>
__device__ __forceinline__ uint4 apply_f32(uint4 xu, float4 nz, unsigned bits, float &m)
{
    const float ninf = -CUDART_INF_F, qnan = CUDART_NAN_F;
    const float x[4] = {__uint_as_float(xu.x), __uint_as_float(xu.y), __uint_as_float(xu.z),
                        __uint_as_float(xu.w)};
    const float add[4] = {nz.x, nz.y, nz.z, nz.w};
    float o[4], c[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const bool ok = bits & (1u << e);
        o[e] = ok ? x[e] : ninf;
        const float s = NOISE ? x[e] + add[e] : x[e];
        c[e] = ok ? s : qnan;
    }
    m = fmaxf(fmaxf(c[0], c[1]), fmaxf(c[2], c[3]));      // fmaxf skips NaN operands
    return make_uint4(__float_as_uint(o[0]), __float_as_uint(o[1]), __float_as_uint(o[2]),
                      __float_as_uint(o[3]));
}

// bf16: 8 logits per 16-byte vector, mask bits in bits[7:0]; noise as two float4.
template <bool NOISE>
__device__ __forceinline__ uint4 apply_bf16(uint4 xu, float4 nza, float4 nzb, unsigned bits,
                                            float &m)
{
    const float qnan = CUDART_NAN_F;
    const unsigned w[4] = {xu.x, xu.y, xu.z, xu.w};
    const float add[8] = {nza.x, nza.y, nza.z, nza.w, nzb.x, nzb.y, nzb.z, nzb.w};
    unsigned o[4];
    float c[8];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const bool ok0 = bits & (1u << (2 * h)), ok1 = bits & (2u << (2 * h));
        const unsigned s0 = ok0 ? w[h] : 0xff80ff80u, s1 = ok1 ? w[h] : 0xff80ff80u;
        o[h] = __byte_perm(s0, s1, 0x7610);               // low half from s0, high half from s1
        float f0 = __uint_as_float(w[h] << 16), f1 = __uint_as_float(w[h] & 0xffff0000u);
        if (NOISE) {
            f0 = f0 + add[2 * h];
            f1 = f1 + add[2 * h + 1];
        }
        c[2 * h] = ok0 ? f0 : qnan;
        c[2 * h + 1] = ok1 ? f1 : qnan;
    }
    m = fmaxf(fmaxf(fmaxf(c[0], c[1]), fmaxf(c[2], c[3])),
              fmaxf(fmaxf(c[4], c[5]), fmaxf(c[6], c[7])));
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// Scalar element, shared by the vector kernel's ragged tail and the scalar kernel.
template <bool BF16>
__device__ __forceinline__ void apply_one(const StepParams &p, const RowCtx &c, long long row_off,
                                          int i, Best &b)
{
    bool ok = false;
    if (!CSTR_INB(p.oob, i, p.V, CSTR_SITE_STEP_LOGITS) ||
        !CSTR_INB(p.oob, row_off + i, (long long)p.batch * p.ld, CSTR_SITE_STEP_LOGITS))
        return;
    if (c.active && CSTR_INB(p.oob, i >> 5, p.tab[c.t].ldw, CSTR_SITE_STEP_MASK))
        ok = (c.mrow[i >> 5] >> (i & 31)) & 1u;
    if (BF16) {
        const unsigned short *in = (const unsigned short *)p.logits + row_off;
        unsigned short *out = (unsigned short *)p.out + row_off;
        const unsigned short raw = in[i];
        float f = __uint_as_float((unsigned)raw << 16);
        if (p.noise && ok)
            f = f + p.noise[row_off + i];
        out[i] = ok ? raw : (unsigned short)0xff80u;
        consider(b, ok ? f : CUDART_NAN_F, i);
    } else {
        const float *in = (const float *)p.logits + row_off;
        float *out = (float *)p.out + row_off;
        const float raw = in[i];
        float f = raw;
        if (p.noise && ok)
            f = f + p.noise[row_off + i];
        out[i] = ok ? raw : -CUDART_INF_F;
        consider(b, ok ? f : CUDART_NAN_F, i);
    }
}

// ---- vector kernel ----------------------------------------------------------

template <bool BF16, bool NOISE, bool PDA>
__global__ void __launch_bounds__(256, 4)
step_vec_kernel(const __grid_constant__ StepParams p)
{
    constexpr int VEC = BF16 ? 8 : 4;               // logits per 16-byte vector
    constexpr int kUnroll = unroll_for(NOISE);
    constexpr int TILE = 32 * VEC * kUnroll;        // tokens per warp tile
    constexpr int WORDS = TILE / 32;                // mask words per tile (16, 32 or 64)
    constexpr int WPL = WORDS >= 32 ? WORDS / 32 : 1;   // mask words per lane per tile
    constexpr int LANES_PER_WORD = 32 / VEC;

    const RowCtx c = row_context<PDA>(p);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const long long row_off = (long long)c.r * p.ld;
    const uint4 *in = (const uint4 *)((const char *)p.logits + row_off * (BF16 ? 2 : 4));
    uint4 *out = (uint4 *)((char *)p.out + row_off * (BF16 ? 2 : 4));
    const float4 *nzrow = NOISE ? (const float4 *)(p.noise + row_off) : nullptr;
    const int total_tiles = (p.V + TILE - 1) / TILE;
    const int tile_end = min(total_tiles, (c.chunk + 1) * p.tiles_per_cta);
    const int Vv = p.V - p.V % VEC;                 // tokens covered by whole vectors

    VBest vb = {-CUDART_INF_F, -1};
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

    for (int tile = c.chunk * p.tiles_per_cta + warp; tile < tile_end; tile += nwarps) {
        const int tok0 = tile * TILE;
        if (!c.active) {                            // finished / invalid row: all -inf
            const uint4 fill = BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                                    : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const int tok = tok0 + (j * 32 + lane) * VEC;
                if (tok < Vv && CSTR_INB(p.oob, row_off + tok + VEC - 1, (long long)p.batch * p.ld,
                                         CSTR_SITE_STEP_LOGITS))
                    __stcs(out + tok / VEC, fill);
            }
            continue;
        }
        uint32_t mw[WPL];
#pragma unroll
        for (int i = 0; i < WPL; ++i) {
            const long long widx = (long long)tile * WORDS + i * 32 + lane;
            // (the bound on widx is part of the kernel: the last tile of a row reaches past W)
            mw[i] = (i * 32 + lane < WORDS && widx < p.tab[c.t].ldw) ? __ldg(c.mrow + widx) : 0u;
        }
        uint4 x[kUnroll];
        float4 nz[NOISE ? kUnroll * (BF16 ? 2 : 1) : 1];
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            const int tok = tok0 + (j * 32 + lane) * VEC;
            x[j] = make_uint4(0u, 0u, 0u, 0u);
            if (tok < Vv && CSTR_INB(p.oob, row_off + tok + VEC - 1, (long long)p.batch * p.ld,
                                     CSTR_SITE_STEP_LOGITS))
                x[j] = __ldcs(in + tok / VEC);
        }
        if (NOISE) {
#pragma unroll
            for (int j = 0; j < kUnroll; ++j) {
                const int tok = tok0 + (j * 32 + lane) * VEC;
                if (BF16) {
                    nz[2 * j] = nz[2 * j + 1] = zero4;
                    if (tok < Vv) {
                        nz[2 * j] = __ldcs(nzrow + tok / 4);
                        nz[2 * j + 1] = __ldcs(nzrow + tok / 4 + 1);
                    }
                } else {
                    nz[j] = zero4;
                    if (tok < Vv)
                        nz[j] = __ldcs(nzrow + tok / 4);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kUnroll; ++j) {
            const int tok = tok0 + (j * 32 + lane) * VEC;
            const int word_in_tile = j * VEC + lane / LANES_PER_WORD;
            const uint32_t word = __shfl_sync(kFull, mw[word_in_tile / 32], word_in_tile % 32);
            const unsigned bits = word >> ((lane % LANES_PER_WORD) * VEC);   // low VEC bits count
            if (tok < Vv) {
                float m;
                uint4 o;
                if (BF16)
                    o = apply_bf16<NOISE>(x[j], NOISE ? nz[2 * j] : zero4,
                                          NOISE ? nz[2 * j + 1] : zero4, bits, m);
                else
                    o = apply_f32<NOISE>(x[j], NOISE ? nz[j] : zero4, bits, m);
                __stcs(out + tok / VEC, o);
                vconsider(vb, m, tok);
            }
        }
    }

    // Winner among the warp's vectors (every lane ends with the same pair), then
    // the element inside that vector: lanes 0..VEC-1 re-read one logit each (an
    // allowed logit is unchanged even when the step runs in place).
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float ov = __shfl_xor_sync(kFull, vb.v, off);
        const int oi = __shfl_xor_sync(kFull, vb.vec, off);
        const bool take = oi >= 0 && (vb.vec < 0 || ov > vb.v || (ov == vb.v && oi < vb.vec));
        vb.v = take ? ov : vb.v;
        vb.vec = take ? oi : vb.vec;
    }
    Best b = {-CUDART_INF_F, -1};
    if (vb.vec >= 0) {                              // warp-uniform
        __syncwarp();
        bool match = false;
        if (lane < VEC && CSTR_INB(p.oob, vb.vec + lane, p.V, CSTR_SITE_STEP_LOGITS)) {
            const int i = vb.vec + lane;
            const bool ok = (c.mrow[i >> 5] >> (i & 31)) & 1u;
            float f;
            if (BF16)
                f = __uint_as_float((unsigned)((const unsigned short *)p.logits)[row_off + i] << 16);
            else
                f = ((const float *)p.logits)[row_off + i];
            if (NOISE)
                f = f + p.noise[row_off + i];
            match = ok && f == vb.v;
        }
        const unsigned hits = __ballot_sync(kFull, match);
        if (hits != 0u && lane == 0) {
            b.v = vb.v;
            b.i = vb.vec + __ffs((int)hits) - 1;
        }
    }
    // ragged tail (V not a multiple of the vector width): highest indices of the row
    if (c.chunk == p.nchunks - 1 && warp == 0 && Vv + lane < p.V) {
        Best tb = {-CUDART_INF_F, -1};
        apply_one<BF16>(p, c, row_off, Vv + lane, tb);
        merge(b, tb.v, tb.i);
    }

    finish_row<PDA>(p, c, b);
}

// ---- scalar kernel: any alignment / stride ----------------------------------

template <bool BF16, bool PDA>
__global__ void __launch_bounds__(256)
step_scalar_kernel(const __grid_constant__ StepParams p)
{
    const RowCtx c = row_context<PDA>(p);
    const long long row_off = (long long)c.r * p.ld;
    const long long begin = (long long)c.chunk * p.tiles_per_cta * p.tile_tokens;
    const int end = (int)min((long long)p.V, begin + (long long)p.tiles_per_cta * p.tile_tokens);
    Best b = {-CUDART_INF_F, -1};
    for (int i = (int)begin + threadIdx.x; i < end; i += blockDim.x)
        apply_one<BF16>(p, c, row_off, i, b);
    finish_row<PDA>(p, c, b);
}

int g_sm_count[64] = {0};

int sm_count(int device)
{
    if (device < 0 || device >= 64)
        return 148;
    if (g_sm_count[device] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n < 1)
            n = 148;
        g_sm_count[device] = n;
    }
    return g_sm_count[device];
}

}  // namespace

int cstr_launch_step(const cstr_step_args &a, cudaStream_t stream)
{
    StepParams p;
    memset(&p, 0, sizeof p);
    for (int i = 0; i < CSTR_MAX_TABLES && !a.pda; ++i) {
        const cstr_table *t = a.tables[i < a.n_tables ? i : 0];
        p.tab[i].mask = t->mask;
        p.tab[i].next = t->next;
        p.tab[i].accept = t->accept;
        p.tab[i].rank = t->renumbered ? t->rank : nullptr;
        p.tab[i].unrank = t->renumbered ? t->unrank : nullptr;
        p.tab[i].lds = t->lds;
        p.tab[i].ldw = t->ldw;
        p.tab[i].n_states = t->n_states;
        p.tab[i].wide = t->wide;
        p.tab[i].code_shift = t->code_shift;
    }
    if (a.pda) {
        p.tab[0].ldw = a.ldw;
        p.pda = *a.pda;
    }
    p.row_mask = a.row_mask;
    p.row_table = a.row_table;
    p.logits = a.logits;
    p.noise = a.noise;
    p.out = a.masked_out;
    p.states = a.states;
    p.states_out = a.states_out;
    p.tokens = a.tokens_out;
    p.accept_out = a.accept_out;
    p.cell = a.cell;
    p.ticket = a.ticket;
    p.counters = a.counters;
    p.ld = a.ld;
    p.V = a.pda ? a.V : a.tables[0]->V;
    p.n_tables = a.n_tables;
    p.batch = a.batch;
    p.oob = CSTR_OOB_RECORD();

    const bool bf16 = a.dtype == CSTR_BF16;
    const int esz = bf16 ? 2 : 4;
    const int tile = 32 * (bf16 ? 8 : 4) * unroll_for(a.noise != nullptr);
    p.tile_tokens = tile;
    const int total_tiles = (p.V + tile - 1) / tile;
    // 16 tiles (two per warp) per CTA when there is enough work to fill the
    // machine a few times over - measured best on B200: one tile per warp leaves
    // the per-warp set-up and reduction dominant, more tiles per CTA unbalance
    // the row tails - and fewer for small batches.
    const long long want_ctas = 4LL * sm_count(a.device);
    int tiles_per_cta = 16;
    while (tiles_per_cta > 1 &&
           (long long)a.batch * ((total_tiles + tiles_per_cta - 1) / tiles_per_cta) < want_ctas)
        tiles_per_cta >>= 1;
    p.tiles_per_cta = tiles_per_cta;
    p.nchunks = (total_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const long long ctas = (long long)a.batch * p.nchunks;
    if (ctas > 0x7fffffffLL)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_step: batch x vocabulary too large for one launch");
    const int threads = 32 * (tiles_per_cta < 8 ? tiles_per_cta : 8);

    auto aligned16 = [](const void *ptr) { return ((uintptr_t)ptr & 15u) == 0; };
    const bool vec_ok = aligned16(a.logits) && aligned16(a.masked_out) &&
                        (a.ld * esz) % 16 == 0 &&
                        (!a.noise || (aligned16(a.noise) && (a.ld * 4) % 16 == 0));
    const unsigned grid = (unsigned)ctas;
    const int variant = (vec_ok ? 4 : 0) | (bf16 ? 2 : 0) | (a.noise ? 1 : 0);
#define CSTR_LAUNCH_STEP(PDA)                                                              \
    switch (variant) {                                                                     \
    case 7: step_vec_kernel<true, true, PDA><<<grid, threads, 0, stream>>>(p); break;      \
    case 6: step_vec_kernel<true, false, PDA><<<grid, threads, 0, stream>>>(p); break;     \
    case 5: step_vec_kernel<false, true, PDA><<<grid, threads, 0, stream>>>(p); break;     \
    case 4: step_vec_kernel<false, false, PDA><<<grid, threads, 0, stream>>>(p); break;    \
    case 3: case 2: step_scalar_kernel<true, PDA><<<grid, threads, 0, stream>>>(p); break; \
    default: step_scalar_kernel<false, PDA><<<grid, threads, 0, stream>>>(p); break;       \
    }
    if (a.pda) {
        CSTR_LAUNCH_STEP(true)
    } else {
        CSTR_LAUNCH_STEP(false)
    }
#undef CSTR_LAUNCH_STEP
    CSTR_CUDA_TRY(cudaGetLastError());
    return CSTR_OK;
}

// ---- speculative decoding: accept / rewind ------------------------------------
//
// After the target model has been penalised and decoded at every drafted
// position (one fused step over batch x (k + 1) rows whose states are the
// draft's state history), each sequence keeps the drafted tokens up to the
// first disagreement, takes the target's token there, and rewinds its
// constraint state to the one that follows that token.

namespace {

__global__ void accept_draft_kernel(const int32_t *__restrict__ draft, const int32_t *__restrict__ tgt_tok,
                                    const int32_t *__restrict__ tgt_state, int k, int batch,
                                    int32_t *__restrict__ n_accepted, int32_t *__restrict__ out_tokens,
                                    int32_t *__restrict__ states)
{
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= batch)
        return;
    const int32_t *d = draft + (long long)r * k;
    const int32_t *t = tgt_tok + (long long)r * (k + 1);
    int n = 0;
    while (n < k && d[n] == t[n])
        ++n;
    for (int i = 0; i <= k; ++i)
        out_tokens[(long long)r * (k + 1) + i] = (i <= n) ? t[i] : -1;
    n_accepted[r] = n;
    states[r] = tgt_state[(long long)r * (k + 1) + n];
}

}  // namespace

int cstr_launch_accept(const int32_t *draft, const int32_t *tgt_tok, const int32_t *tgt_state,
                       int32_t k, int32_t batch, int32_t *n_accepted, int32_t *out_tokens,
                       int32_t *states, cudaStream_t stream)
{
    accept_draft_kernel<<<(batch + 127) / 128, 128, 0, stream>>>(draft, tgt_tok, tgt_state, k, batch,
                                                                  n_accepted, out_tokens, states);
    CSTR_CUDA_TRY(cudaGetLastError());
    return CSTR_OK;
}

// ---- allocation-free variant -------------------------------------------------
//
// Same kernels, but the per-row scratch (cells, tickets, counters) lives in one
// fixed array that is part of the loaded library image, so the call never asks
// the CUDA allocator for anything.

namespace {

constexpr int kStaticRows = CSTR_STATIC_MAX_BATCH;
// [0, kStaticRows) cells (u64) | tickets (u32, two per u64) | 2 counters
constexpr size_t kStaticWords = (size_t)kStaticRows + (size_t)kStaticRows / 2 + 2;

static __device__ __align__(256) unsigned long long g_static_scratch[kStaticWords];

// Device address of g_static_scratch per device, resolved on first use.  In
// host code the symbol's name is only a handle for the runtime, not a device
// address, so it must never be passed to a kernel directly.
std::mutex g_static_mutex;
unsigned long long *g_static_ptr[64] = {nullptr};

}  // namespace

extern "C" int cstr_step_static(const cstr_table_t *const *tables, int32_t n_tables,
                                const int32_t *row_table, const void *logits, int32_t dtype,
                                int64_t ld, const float *noise, int32_t *states,
                                int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                                int32_t batch, void *cuda_stream)
{
    if (batch == 0 && tables && (dtype == CSTR_F32 || dtype == CSTR_BF16))
        return CSTR_OK;              // nothing to do: the per-row arrays may be empty (null)
    if (!tables || !logits || !states || !tokens_out || !masked_out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_step_static: null pointer");
    if (n_tables < 1 || n_tables > CSTR_MAX_TABLES)
        return cstr_fail(CSTR_ERR_ARG, "cstr_step_static: n_tables = %d, need 1..%d", n_tables,
                         CSTR_MAX_TABLES);
    if (dtype != CSTR_F32 && dtype != CSTR_BF16)
        return cstr_fail(CSTR_ERR_DTYPE, "cstr_step_static: unknown dtype %d", dtype);
    if (batch < 0)
        return cstr_fail(CSTR_ERR_ARG, "cstr_step_static: batch = %d", batch);
    if (batch > kStaticRows)
        return cstr_fail(CSTR_ERR_SHAPE,
                         "cstr_step_static: batch %d exceeds the built-in scratch of %d rows; "
                         "use cstr_step with a workspace for larger batches",
                         batch, kStaticRows);
    int device = -1;
    CSTR_CUDA_TRY(cudaGetDevice(&device));
    if (device < 0 || device >= 64)
        return cstr_fail(CSTR_ERR_DEVICE, "cstr_step_static: device index %d not supported", device);
    cstr_step_args a;
    memset(&a, 0, sizeof a);
    for (int32_t i = 0; i < n_tables; ++i) {
        const cstr_table *t = tables[i];
        if (!t)
            return cstr_fail(CSTR_ERR_NULL, "cstr_step_static: tables[%d] is null", i);
        if (t->device != device)
            return cstr_fail(CSTR_ERR_DEVICE, "cstr_step_static: tables[%d] is on device %d, "
                             "device %d is current", i, t->device, device);
        if (t->n_states < 1)
            return cstr_fail(CSTR_ERR_ARG, "cstr_step_static: tables[%d] has not been built", i);
        if (t->V != tables[0]->V)
            return cstr_fail(CSTR_ERR_SHAPE, "cstr_step_static: tables[%d] has V = %d, "
                             "tables[0] has %d", i, t->V, tables[0]->V);
        a.tables[i] = t;
    }
    if (ld < tables[0]->V)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_step_static: ld = %lld is below V = %d",
                         (long long)ld, tables[0]->V);
    if (batch == 0)
        return CSTR_OK;

    unsigned long long *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[device]) {
            void *ptr = nullptr;
            cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e != cudaSuccess || !ptr)
                return cstr_fail(CSTR_ERR_CUDA, "cstr_step_static: cudaGetSymbolAddress: %s",
                                 cudaGetErrorString(e));
            g_static_ptr[device] = (unsigned long long *)ptr;
        }
        scratch = g_static_ptr[device];
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // The array keeps whatever the previous call (or an interrupted one) left.
    CSTR_CUDA_TRY(cudaMemsetAsync(scratch, 0, kStaticWords * sizeof(unsigned long long), stream));

    a.n_tables = n_tables;
    a.row_table = row_table;
    a.logits = logits;
    a.dtype = dtype;
    a.ld = ld;
    a.noise = noise;
    a.states = states;
    a.states_out = states;
    a.tokens_out = tokens_out;
    a.masked_out = masked_out;
    a.accept_out = accept_out;
    a.batch = batch;
    a.cell = scratch;
    a.ticket = (unsigned int *)(scratch + kStaticRows);
    a.counters = scratch + kStaticRows + kStaticRows / 2;
    a.device = device;
    return cstr_launch_step(a, stream);
}
