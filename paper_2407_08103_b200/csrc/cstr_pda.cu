// Push-down constraints (Section 3; Algorithm 3): the token-level PDA
// P_{G o V} = P_G o T_V in a dense per-situation form, and the batched decoding
// step that keeps a state and a stack per row.
//
// An edge of P_{G o V} reads a token by chaining the byte edges of its
// characters, so what it pops depends on how far the chain reaches into the
// stack it finds.  For all but a handful of tokens the top symbol is enough, so
// the table keeps, per situation (state q, top symbol X or "empty"), one row of
// allowed-token bits decided with X alone, and a second row flagging the tokens
// whose fate depends on deeper symbols.  At decode time a row takes its
// situation's mask row as is, or - if that situation has flagged tokens - a
// private copy in which the flagged tokens have been walked against the row's
// real stack.  The fused step kernel then streams the logits exactly as in the
// finite-state case, and the last CTA of each row traverses the selected
// token's edge: it walks the token's bytes from (q, s), which yields the edge's
// target, pops and pushes without storing variable-length stack edits per
// table entry.
#include <string.h>

#include <new>
#include <vector>

#include "cstr_internal.cuh"
#include "cstr_pda_walk.cuh"

namespace {

using namespace cstr_pda_dev;

// The table is built in two passes.  Most walks never look at the stack, so a
// first pass decides every (state, token) pair with the top of the stack
// unknown: allowed whatever the stack holds, dead, or "looks at the top".  The
// second pass fills the rows of the situations (state, top): it copies the
// state's stack-independent bits and walks only the tokens of the third kind,
// now with the top known.  One warp per 32-token word, lane = token.
__global__ void __launch_bounds__(256)
pda_state_pass_kernel(cstr_pda_view P, const uint8_t *__restrict__ accept,
                      const uint8_t *__restrict__ vbytes, const uint32_t *__restrict__ voff, int V,
                      int W, long long ldw, int eos_id, uint32_t *__restrict__ base,
                      uint32_t *__restrict__ need)
{
    const int lane = threadIdx.x & 31;
    const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int q = blockIdx.y;
    if (w >= W)
        return;
    const int v = w * 32 + lane;
    int res = WALK_DEAD;
    if (v < V) {
        if (v == eos_id) {
            res = accept[q] ? WALK_OK : WALK_DEAD;
        } else {
            uint8_t loc[kLocMax];
            int q2, cd2, nloc2;
            const uint32_t b = voff[v], e = voff[v + 1];
            res = pda_walk(P, q, nullptr, 0, 0, true, vbytes + b, (int)(e - b), loc, q2, cd2, nloc2);
        }
    }
    const unsigned ok = __ballot_sync(0xffffffffu, res == WALK_OK);
    const unsigned nd = __ballot_sync(0xffffffffu, res == WALK_DEEP);
    if (lane == 0) {
        base[(long long)q * ldw + w] = ok;
        need[(long long)q * ldw + w] = nd;
    }
}

// One warp per 32 consecutive words of a situation's rows: lane = word for the
// (coalesced) copy; for the few words that hold top-dependent tokens the whole
// warp walks that word's tokens, lane = token.
__global__ void __launch_bounds__(256)
pda_situation_pass_kernel(cstr_pda_view P, const uint8_t *__restrict__ vbytes,
                          const uint32_t *__restrict__ voff, long long ldw,
                          const uint32_t *__restrict__ base, const uint32_t *__restrict__ need,
                          uint32_t *__restrict__ mask, uint32_t *__restrict__ deep,
                          uint32_t *__restrict__ ndeep)
{
    const int lane = threadIdx.x & 31;
    const long long w0 = ((long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * 32;
    const int cfg = blockIdx.y;
    if (w0 >= ldw)
        return;                                     // ldw is a multiple of 32: whole groups
    const int q = cfg / (P.n_symbols + 1);
    const int top = cfg - q * (P.n_symbols + 1);    // n_symbols = empty stack
    const bool has_top = top < P.n_symbols;
    unsigned ok = base[(long long)q * ldw + w0 + lane];
    const unsigned nd = need[(long long)q * ldw + w0 + lane];
    unsigned dp = 0u;
    unsigned pending = __ballot_sync(0xffffffffu, nd != 0u);
    while (pending) {                               // warp-uniform
        const int src = __ffs((int)pending) - 1;
        pending &= pending - 1;
        const unsigned word_nd = __shfl_sync(0xffffffffu, nd, src);
        int res = WALK_DEAD;
        if ((word_nd >> lane) & 1u) {
            const int v = (int)(w0 + src) * 32 + lane;
            uint8_t loc[kLocMax];
            int q2, cd2, nloc2;
            const uint32_t b = voff[v], e = voff[v + 1];
            res = pda_walk(P, q, nullptr, top, has_top ? 1 : 0, has_top, vbytes + b, (int)(e - b),
                           loc, q2, cd2, nloc2);
        }
        const unsigned got_ok = __ballot_sync(0xffffffffu, res == WALK_OK);
        const unsigned got_dp = __ballot_sync(0xffffffffu, res == WALK_DEEP);
        if (lane == src) {
            ok |= got_ok;
            dp = got_dp;
        }
    }
    mask[(long long)cfg * ldw + w0 + lane] = ok;
    deep[(long long)cfg * ldw + w0 + lane] = dp;
    const unsigned total = __reduce_add_sync(0xffffffffu, (unsigned)__popc(dp));
    if (lane == 0 && total)
        atomicAdd(ndeep + cfg, total);
}

// What the prepare kernel reads: the rows' situations and the table.
struct PdaPrepParams {
    cstr_pda_view P;
    const uint8_t *vbytes;
    const uint32_t *voff;
    const uint32_t *mask, *deep, *ndeep;
    long long ldw;
    int n_states;
    const int32_t *states, *stacks, *depths;
    int cap;
    const uint32_t **row_mask;
    uint32_t *row_buf;
};

// Find each row's situation and point the step at its mask row, or - when the
// situation has tokens that depend on deeper stack symbols - at a private copy
// in which those tokens have been walked against the row's real stack.
// blockIdx.x = row, blockIdx.y = slice of kPrepWords mask words; every block of
// a row re-derives the (cheap) row checks.
constexpr int kPrepThreads = 256;
constexpr int kPrepWords = 1024;

__global__ void __launch_bounds__(kPrepThreads)
pda_prepare_kernel(const __grid_constant__ PdaPrepParams p)
{
    const int r = blockIdx.x;
    const int slice = blockIdx.y;
    const int q = p.states[r];
    const int d = p.depths[r];
    const int32_t *s = p.stacks + (long long)r * p.cap;
    const bool shape_ok = q >= 0 && q < p.n_states && d >= 0 && d <= p.cap;   // block-uniform
    bool bad = false;
    if (shape_ok)
        for (int i = threadIdx.x; i < d; i += kPrepThreads)
            bad |= (unsigned)s[i] >= (unsigned)p.P.n_symbols;
    const bool ok = shape_ok && !__syncthreads_or(bad);
    if (!ok) {
        if (slice == 0 && threadIdx.x == 0)
            p.row_mask[r] = nullptr;
        return;
    }
    const int top = d > 0 ? s[d - 1] : p.P.n_symbols;
    const long long cfg = (long long)q * (p.P.n_symbols + 1) + top;
    const uint32_t *mrow = p.mask + cfg * p.ldw;
    if (p.ndeep[cfg] == 0) {
        if (slice == 0 && threadIdx.x == 0)
            p.row_mask[r] = mrow;
        return;
    }
    const uint32_t *drow = p.deep + cfg * p.ldw;
    uint32_t *out = p.row_buf + (long long)r * p.ldw;
    // Pass 1: copy the words without flagged tokens, queue the others.
    __shared__ int s_queue[kPrepWords];
    __shared__ int s_count;
    if (threadIdx.x == 0)
        s_count = 0;
    __syncthreads();
    constexpr int kPer = kPrepWords / kPrepThreads;
    const long long w0 = (long long)slice * kPrepWords + threadIdx.x;
    uint32_t mw[kPer], dw[kPer];
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const long long w = w0 + (long long)j * kPrepThreads;
        mw[j] = w < p.ldw ? __ldg(mrow + w) : 0u;
        dw[j] = w < p.ldw ? __ldg(drow + w) : 0u;
    }
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const long long w = w0 + (long long)j * kPrepThreads;
        if (w >= p.ldw)
            continue;
        if (dw[j] == 0u)
            out[w] = mw[j];
        else
            s_queue[atomicAdd(&s_count, 1)] = (int)w;
    }
    __syncthreads();
    // Pass 2: one warp per queued word, one lane per flagged token - each walk is
    // a chain of dependent loads, so the tokens of a word are walked side by side.
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = warp; i < s_count; i += kPrepThreads / 32) {
        const long long w = s_queue[i];
        const uint32_t flagged = __ldg(drow + w);
        bool allowed = false;
        if ((flagged >> lane) & 1u) {
            const int v = (int)w * 32 + lane;
            uint8_t loc[kLocMax];
            int q2, cd2, nloc2;
            const uint32_t b0 = p.voff[v], b1 = p.voff[v + 1];
            allowed = pda_walk(p.P, q, s, 0, d, false, p.vbytes + b0, (int)(b1 - b0), loc, q2, cd2,
                               nloc2) == WALK_OK;
        }
        const uint32_t extra = __ballot_sync(0xffffffffu, allowed);
        if (lane == 0)
            out[w] = __ldg(mrow + w) | extra;
    }
    if (slice == 0 && threadIdx.x == 0)
        p.row_mask[r] = out;
}

int cuda_rc(cudaError_t e, const char *who)
{
    return cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA, "%s: %s", who,
                     cudaGetErrorString(e));
}

}  // namespace

// ------------------------------------------------------------------ PDA

extern "C" void cstr_free_pda(cstr_pda_t *p)
{
    if (!p)
        return;
    cudaFree(p->act);
    cudaFree(p->edge);
    cudaFree(p->accept);
    delete p;
}

extern "C" int cstr_load_pda(const int32_t *edge_src, const int32_t *edge_byte,
                             const int32_t *edge_tgt, const int32_t *pop_off, const int32_t *pops,
                             const int32_t *push_off, const int32_t *pushes, int32_t n_edges,
                             const uint8_t *accept, int32_t n_states, int32_t n_symbols,
                             int32_t start_state, cstr_pda_t **out)
{
    if (!out || !accept || !pop_off || !push_off ||
        (n_edges > 0 && (!edge_src || !edge_byte || !edge_tgt)))
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_pda: null pointer");
    *out = nullptr;
    if (n_states < 1 || n_edges < 0)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_pda: n_states = %d, n_edges = %d", n_states,
                         n_edges);
    if (n_symbols < 0 || n_symbols > CSTR_PDA_MAX_SYMBOLS)
        return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: n_symbols = %d, need 0..%d", n_symbols,
                         CSTR_PDA_MAX_SYMBOLS);
    if (start_state < 0 || start_state >= n_states)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_pda: start_state %d outside [0, %d)",
                         start_state, n_states);
    const int NT = n_symbols + 2;
    const int64_t slots = (int64_t)n_states * NT * 256;
    if (slots > ((int64_t)1 << 28))
        return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: %d states x %d symbols exceed the lookup "
                         "table limit of 2^28 entries", n_states, n_symbols);
    if (pop_off[0] != 0 || push_off[0] != 0)
        return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: pop_off[0] and push_off[0] must be 0");

    std::vector<uint32_t> act;
    std::vector<int2> edges;
    std::vector<uint8_t> flags;
    int max_push = 0;
    try {
        act.assign((size_t)slots, CSTR_PDA_NONE);
        edges.resize((size_t)n_edges);
        flags.resize((size_t)n_states);
    } catch (const std::bad_alloc &) {
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_pda: out of host memory");
    }
    for (int32_t q = 0; q < n_states; ++q)
        flags[q] = accept[q] ? 1 : 0;
    for (int32_t j = 0; j < n_edges; ++j) {
        const int32_t q = edge_src[j], b = edge_byte[j], t = edge_tgt[j];
        if (q < 0 || q >= n_states || t < 0 || t >= n_states)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d joins states %d -> %d outside "
                             "[0, %d)", j, q, t, n_states);
        if (b < 0 || b > 255)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d reads %d; every edge must read "
                             "one byte 0..255 (no epsilon input)", j, b);
        const int32_t np = pop_off[j + 1] - pop_off[j], nu = push_off[j + 1] - push_off[j];
        if (np < 0 || nu < 0)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: offsets decrease at edge %d", j);
        if (np > 1)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d pops %d symbols, at most 1 "
                             "supported", j, np);
        if (nu > CSTR_PDA_MAX_PUSH)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d pushes %d symbols, at most %d "
                             "supported", j, nu, CSTR_PDA_MAX_PUSH);
        if ((np > 0 && !pops) || (nu > 0 && !pushes))
            return cstr_fail(CSTR_ERR_NULL, "cstr_load_pda: null pops / pushes");
        unsigned meta = (unsigned)nu << 24 | (unsigned)np << 28;
        for (int32_t i = 0; i < nu; ++i) {
            const int32_t y = pushes[push_off[j] + i];
            if (y < 0 || y >= n_symbols)
                return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d pushes symbol %d outside "
                                 "[0, %d)", j, y, n_symbols);
            meta |= (unsigned)y << (8 * i);
        }
        if (nu > max_push)
            max_push = nu;
        edges[j] = make_int2(t, (int)meta);
        uint32_t *row = act.data() + (size_t)q * NT * 256 + b;   // row[t * 256]
        bool clash = false;
        if (np == 0) {
            for (int tt = 0; tt < NT; ++tt) {
                clash |= row[(size_t)tt * 256] != CSTR_PDA_NONE;
                row[(size_t)tt * 256] = (uint32_t)j;
            }
        } else {
            const int32_t x = pops[pop_off[j]];
            if (x < 0 || x >= n_symbols)
                return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: edge %d pops symbol %d outside "
                                 "[0, %d)", j, x, n_symbols);
            uint32_t &unknown = row[(size_t)(n_symbols + 1) * 256];
            clash = row[(size_t)x * 256] != CSTR_PDA_NONE ||
                    (unknown != CSTR_PDA_NONE && unknown != CSTR_PDA_NEEDCTX);
            row[(size_t)x * 256] = (uint32_t)j;
            unknown = CSTR_PDA_NEEDCTX;
        }
        if (clash)
            return cstr_fail(CSTR_ERR_PDA, "cstr_load_pda: not deterministic: edge %d (state %d, "
                             "byte %d) competes with an earlier edge", j, q, b);
    }

    cstr_pda *p = new (std::nothrow) cstr_pda();
    if (!p)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_pda: out of host memory");
    memset(p, 0, sizeof *p);
    p->n_states = n_states;
    p->n_symbols = n_symbols;
    p->start = start_state;
    p->n_edges = n_edges;
    p->NT = NT;
    p->max_push = max_push;
    cudaError_t e = cudaGetDevice(&p->device);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&p->act, (size_t)slots * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&p->edge, ((size_t)n_edges + 1) * sizeof(int2));
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&p->accept, (size_t)n_states);
    if (e == cudaSuccess)
        e = cudaMemcpy(p->act, act.data(), (size_t)slots * 4, cudaMemcpyHostToDevice);
    if (e == cudaSuccess && n_edges > 0)
        e = cudaMemcpy(p->edge, edges.data(), (size_t)n_edges * sizeof(int2),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(p->accept, flags.data(), (size_t)n_states, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        const int rc = cuda_rc(e, "cstr_load_pda");
        cstr_free_pda(p);
        return rc;
    }
    *out = p;
    return CSTR_OK;
}

// ---------------------------------------------------------------- table

extern "C" void cstr_free_pda_table(cstr_pda_table_t *t)
{
    if (!t)
        return;
    cudaFree(t->mask);
    cudaFree(t->deep);
    cudaFree(t->ndeep);
    cudaFree(t->base);
    cudaFree(t->need);
    delete t;
}

// The two build passes into a table's existing storage (every word of the
// situation rows is rewritten; only the per-situation counts need clearing).
static cudaError_t enqueue_pda_build(cstr_pda_table *t, cudaStream_t stream)
{
    const cstr_pda *pda = t->pda;
    const cstr_vocab *vocab = t->vocab;
    cudaError_t e = cudaMemsetAsync(t->ndeep, 0, (size_t)t->n_cfg * 4, stream);
    if (e != cudaSuccess)
        return e;
    cstr_pda_view P = {pda->act, pda->edge, pda->NT, pda->n_symbols,
                       (long long)pda->n_states * pda->NT * 256, pda->n_edges, CSTR_OOB_RECORD()};
    const int warps = 8;
    const unsigned gx = (unsigned)((t->W + warps - 1) / warps);
    pda_state_pass_kernel<<<dim3(gx, (unsigned)pda->n_states), warps * 32, 0, stream>>>(
        P, pda->accept, vocab->bytes, vocab->off, t->V, t->W, t->ldw, t->eos_id, t->base, t->need);
    const unsigned gx2 = (unsigned)((t->ldw / 32 + warps - 1) / warps);
    pda_situation_pass_kernel<<<dim3(gx2, (unsigned)t->n_cfg), warps * 32, 0, stream>>>(
        P, vocab->bytes, vocab->off, t->ldw, t->base, t->need, t->mask, t->deep, t->ndeep);
    return cudaGetLastError();
}

extern "C" int cstr_pda_table_rebuild(cstr_pda_table_t *t, int32_t eos_id, void *cuda_stream)
{
    if (!t)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_table_rebuild: null table");
    int rc = cstr_check_device(t->device, "PDA table");
    if (rc)
        return rc;
    if (eos_id < -1 || eos_id >= t->V)
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_table_rebuild: eos_id %d outside [-1, %d)", eos_id,
                         t->V);
    t->eos_id = eos_id;
    const cudaError_t e = enqueue_pda_build(t, (cudaStream_t)cuda_stream);
    if (e != cudaSuccess)
        return cuda_rc(e, "cstr_pda_table_rebuild");
    return CSTR_OK;
}

extern "C" int cstr_build_pda_table(const cstr_pda_t *pda, const cstr_vocab_t *vocab,
                                    int32_t eos_id, void *cuda_stream, cstr_pda_table_t **out)
{
    if (!pda || !vocab || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_build_pda_table: null pointer");
    *out = nullptr;
    int rc = cstr_check_device(pda->device, "PDA");
    if (rc)
        return rc;
    if (vocab->device != pda->device)
        return cstr_fail(CSTR_ERR_DEVICE, "cstr_build_pda_table: PDA and vocabulary on different "
                         "devices");
    if (eos_id < -1 || eos_id >= vocab->V)
        return cstr_fail(CSTR_ERR_ARG, "cstr_build_pda_table: eos_id %d outside [-1, %d)", eos_id,
                         vocab->V);
    if ((int64_t)vocab->max_len * (pda->max_push > 0 ? pda->max_push : 1) > kLocMax - 1)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_build_pda_table: a token of %u bytes with edges "
                         "that push up to %d symbols could leave more than %d symbols",
                         vocab->max_len, pda->max_push, kLocMax - 1);
    cstr_pda_table *t = new (std::nothrow) cstr_pda_table();
    if (!t)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_build_pda_table: out of host memory");
    memset(t, 0, sizeof *t);
    t->device = pda->device;
    t->pda = pda;
    t->vocab = vocab;
    t->V = vocab->V;
    t->W = (vocab->V + 31) / 32;
    t->ldw = ((int64_t)t->W + 31) / 32 * 32;
    t->eos_id = eos_id;
    const int64_t n_cfg = (int64_t)pda->n_states * (pda->n_symbols + 1);
    if (n_cfg > 65535) {
        delete t;
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_build_pda_table: %lld (state, top) situations, at "
                         "most 65535 supported", (long long)n_cfg);
    }
    t->n_cfg = (int32_t)n_cfg;
    const size_t row_bytes = (size_t)n_cfg * (size_t)t->ldw * 4;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    cudaError_t e = cudaMalloc((void **)&t->mask, row_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->deep, row_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->ndeep, (size_t)n_cfg * 4);
    const size_t state_bytes = (size_t)pda->n_states * (size_t)t->ldw * 4;
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->base, state_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->need, state_bytes);
    if (e == cudaSuccess)
        e = cudaMemsetAsync(t->base, 0, state_bytes, stream);   // padding words stay zero
    if (e == cudaSuccess)
        e = cudaMemsetAsync(t->need, 0, state_bytes, stream);
    if (e == cudaSuccess)
        e = enqueue_pda_build(t, stream);
    if (e != cudaSuccess) {
        rc = cuda_rc(e, "cstr_build_pda_table");
        cstr_free_pda_table(t);
        return rc;
    }
    *out = t;
    return CSTR_OK;
}

extern "C" int cstr_pda_table_info(const cstr_pda_table_t *t, int32_t *n_states,
                                   int32_t *n_symbols, int32_t *vocab_size, int32_t *mask_words,
                                   int32_t *start_state)
{
    if (!t)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_table_info: null table");
    if (n_states)
        *n_states = t->pda->n_states;
    if (n_symbols)
        *n_symbols = t->pda->n_symbols;
    if (vocab_size)
        *vocab_size = t->V;
    if (mask_words)
        *mask_words = t->W;
    if (start_state)
        *start_state = t->pda->start;
    return CSTR_OK;
}

extern "C" int cstr_pda_table_download(const cstr_pda_table_t *t, int32_t state, int32_t top,
                                       uint32_t *mask_host, uint32_t *deep_host, void *cuda_stream)
{
    if (!t)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_table_download: null table");
    int rc = cstr_check_device(t->device, "PDA table");
    if (rc)
        return rc;
    if (state < 0 || state >= t->pda->n_states || top < -1 || top >= t->pda->n_symbols)
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_table_download: (state %d, top %d) outside "
                         "[0, %d) x [-1, %d)", state, top, t->pda->n_states, t->pda->n_symbols);
    CSTR_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    const int64_t cfg = (int64_t)state * (t->pda->n_symbols + 1) + (top < 0 ? t->pda->n_symbols : top);
    if (mask_host)
        CSTR_CUDA_TRY(cudaMemcpy(mask_host, t->mask + cfg * t->ldw, (size_t)t->W * 4,
                                 cudaMemcpyDeviceToHost));
    if (deep_host)
        CSTR_CUDA_TRY(cudaMemcpy(deep_host, t->deep + cfg * t->ldw, (size_t)t->W * 4,
                                 cudaMemcpyDeviceToHost));
    return CSTR_OK;
}

// ------------------------------------------------------------ workspace

extern "C" void cstr_free_pda_workspace(cstr_pda_workspace_t *ws)
{
    if (!ws)
        return;
    cudaFree(ws->cell);
    cudaFree(ws->ticket);
    cudaFree(ws->counters);
    cudaFree((void *)ws->row_mask);
    cudaFree(ws->row_buf);
    delete ws;
}

extern "C" int cstr_pda_workspace_create(const cstr_pda_table_t *table, int32_t max_batch,
                                         cstr_pda_workspace_t **out)
{
    if (!table || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_workspace_create: null pointer");
    *out = nullptr;
    if (max_batch < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_workspace_create: max_batch = %d, need >= 1",
                         max_batch);
    int rc = cstr_check_device(table->device, "PDA table");
    if (rc)
        return rc;
    cstr_pda_workspace *ws = new (std::nothrow) cstr_pda_workspace();
    if (!ws)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_pda_workspace_create: out of host memory");
    memset(ws, 0, sizeof *ws);
    ws->device = table->device;
    ws->max_batch = max_batch;
    ws->ldw = table->ldw;
    const size_t buf_bytes = (size_t)max_batch * (size_t)ws->ldw * 4;
    cudaError_t e = cudaMalloc((void **)&ws->cell, (size_t)max_batch * 8);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->ticket, (size_t)max_batch * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->counters, 5 * 8);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->row_mask, (size_t)max_batch * sizeof(void *));
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->row_buf, buf_bytes);
    if (e == cudaSuccess)
        e = cudaMemset(ws->cell, 0, (size_t)max_batch * 8);
    if (e == cudaSuccess)
        e = cudaMemset(ws->ticket, 0, (size_t)max_batch * 4);
    if (e == cudaSuccess)
        e = cudaMemset(ws->counters, 0, 5 * 8);
    if (e == cudaSuccess)
        e = cudaMemset((void *)ws->row_mask, 0, (size_t)max_batch * sizeof(void *));
    if (e != cudaSuccess) {
        rc = cuda_rc(e, "cstr_pda_workspace_create");
        cstr_free_pda_workspace(ws);
        return rc;
    }
    *out = ws;
    return CSTR_OK;
}

// ----------------------------------------------------------------- step

static int pda_step_common(const cstr_pda_table_t *table, const void *logits, int32_t dtype,
                           int64_t ld, const float *noise, const int32_t *states_in,
                           const int32_t *stacks_in, const int32_t *depths_in, int32_t *states,
                           int32_t *stacks, int32_t *depths, int32_t stack_cap, int32_t *tokens_out,
                           void *masked_out, uint8_t *accept_out, int32_t batch,
                           cstr_pda_workspace_t *ws, void *cuda_stream)
{
    if (batch == 0 && table && ws && (dtype == CSTR_F32 || dtype == CSTR_BF16) && stack_cap >= 1)
        return CSTR_OK;              // nothing to do: the per-row arrays may be empty (null)
    if (!table || !logits || !states || !stacks || !depths || !states_in || !stacks_in ||
        !depths_in || !tokens_out || !masked_out || !ws)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_step: null pointer");
    if ((stacks_in == stacks) != (depths_in == depths) || (stacks_in == stacks) != (states_in == states))
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_step_history: states, stacks and depths must be "
                         "either all updated in place or all written to separate arrays");
    if (dtype != CSTR_F32 && dtype != CSTR_BF16)
        return cstr_fail(CSTR_ERR_DTYPE, "cstr_pda_step: unknown dtype %d", dtype);
    if (batch < 0 || stack_cap < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_step: batch = %d, stack_cap = %d", batch,
                         stack_cap);
    if (batch > ws->max_batch || ws->ldw != table->ldw)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_pda_step: workspace holds %d rows of %lld words, "
                         "the call needs %d rows of %lld", ws->max_batch, (long long)ws->ldw, batch,
                         (long long)table->ldw);
    if (ld < table->V)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_pda_step: ld = %lld is below V = %d", (long long)ld,
                         table->V);
    int rc = cstr_check_device(ws->device, "PDA workspace");
    if (rc)
        return rc;
    if (table->device != ws->device)
        return cstr_fail(CSTR_ERR_DEVICE, "cstr_pda_step: table is on another device");
    if (batch == 0)
        return CSTR_OK;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    const cstr_pda *pda = table->pda;

    PdaPrepParams p;
    memset(&p, 0, sizeof p);
    p.P.act = pda->act;
    p.P.edge = pda->edge;
    p.P.NT = pda->NT;
    p.P.n_symbols = pda->n_symbols;
    p.P.act_len = (long long)pda->n_states * pda->NT * 256;
    p.P.n_edges = pda->n_edges;
    p.P.oob = CSTR_OOB_RECORD();
    p.vbytes = table->vocab->bytes;
    p.voff = table->vocab->off;
    p.mask = table->mask;
    p.deep = table->deep;
    p.ndeep = table->ndeep;
    p.ldw = table->ldw;
    p.n_states = pda->n_states;
    p.states = states_in;
    p.stacks = stacks_in;
    p.depths = depths_in;
    p.cap = stack_cap;
    p.row_mask = ws->row_mask;
    p.row_buf = ws->row_buf;

    const long long slices = (table->ldw + kPrepWords - 1) / kPrepWords;
    if (slices > 65535)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_pda_step: vocabulary too large");
    pda_prepare_kernel<<<dim3((unsigned)batch, (unsigned)slices), kPrepThreads, 0, stream>>>(p);
    CSTR_CUDA_TRY(cudaGetLastError());

    cstr_step_args a;
    memset(&a, 0, sizeof a);
    a.n_tables = 1;
    a.logits = logits;
    a.dtype = dtype;
    a.ld = ld;
    a.noise = noise;
    a.states = states_in;
    a.states_out = states;
    a.tokens_out = tokens_out;
    a.masked_out = masked_out;
    a.batch = batch;
    a.cell = ws->cell;
    a.ticket = ws->ticket;
    a.counters = ws->counters;
    a.device = ws->device;
    cstr_pda_advance adv;
    memset(&adv, 0, sizeof adv);
    adv.P = p.P;
    adv.accept = pda->accept;
    adv.vbytes = p.vbytes;
    adv.voff = p.voff;
    adv.n_states = pda->n_states;
    adv.eos_id = table->eos_id;
    adv.cap = stack_cap;
    adv.states_in = states_in;
    adv.stacks_in = stacks_in;
    adv.depths_in = depths_in;
    adv.states = states;
    adv.stacks = stacks;
    adv.depths = depths;
    adv.accept_out = accept_out;
    adv.counters = ws->counters + 2;
    a.pda = &adv;
    a.row_mask = ws->row_mask;
    a.V = table->V;
    a.ldw = table->ldw;
    return cstr_launch_step(a, stream);
}

extern "C" int cstr_pda_step(const cstr_pda_table_t *table, const void *logits, int32_t dtype,
                             int64_t ld, const float *noise, int32_t *states, int32_t *stacks,
                             int32_t *depths, int32_t stack_cap, int32_t *tokens_out,
                             void *masked_out, uint8_t *accept_out, int32_t batch,
                             cstr_pda_workspace_t *ws, void *cuda_stream)
{
    return pda_step_common(table, logits, dtype, ld, noise, states, stacks, depths, states, stacks,
                           depths, stack_cap, tokens_out, masked_out, accept_out, batch, ws,
                           cuda_stream);
}

extern "C" int cstr_pda_step_history(const cstr_pda_table_t *table, const void *logits,
                                     int32_t dtype, int64_t ld, const float *noise,
                                     const int32_t *states_in, const int32_t *stacks_in,
                                     const int32_t *depths_in, int32_t *states_out,
                                     int32_t *stacks_out, int32_t *depths_out, int32_t stack_cap,
                                     int32_t *tokens_out, void *masked_out, uint8_t *accept_out,
                                     int32_t batch, cstr_pda_workspace_t *ws, void *cuda_stream)
{
    return pda_step_common(table, logits, dtype, ld, noise, states_in, stacks_in, depths_in,
                           states_out, stacks_out, depths_out, stack_cap, tokens_out, masked_out,
                           accept_out, batch, ws, cuda_stream);
}

// ---- speculative decoding: accept / rewind --------------------------------------
//
// As in the finite-state case, but the constraint's situation after a token is
// a state plus a stack, so the history holds all three per drafted position and
// the rewind copies the stack of the position it goes back to.

namespace {

__global__ void __launch_bounds__(128)
pda_accept_draft_kernel(const int32_t *__restrict__ draft, const int32_t *__restrict__ tgt_tok,
                        const int32_t *__restrict__ tgt_state, const int32_t *__restrict__ tgt_stacks,
                        const int32_t *__restrict__ tgt_depth, int k, int batch, int cap,
                        int32_t *__restrict__ n_accepted, int32_t *__restrict__ out_tokens,
                        int32_t *__restrict__ states, int32_t *__restrict__ stacks,
                        int32_t *__restrict__ depths)
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
    const long long at = (long long)r * (k + 1) + n;
    states[r] = tgt_state[at];
    const int depth = tgt_depth[at];
    depths[r] = depth;
    const int32_t *src = tgt_stacks + at * cap;
    int32_t *dst = stacks + (long long)r * cap;
    for (int i = 0; i < depth && i < cap; ++i)
        dst[i] = src[i];
}

}  // namespace

extern "C" int cstr_pda_accept_draft(const int32_t *draft_tokens, const int32_t *target_tokens,
                                     const int32_t *target_states, const int32_t *target_stacks,
                                     const int32_t *target_depths, int32_t k, int32_t batch,
                                     int32_t stack_cap, int32_t *n_accepted, int32_t *out_tokens,
                                     int32_t *states, int32_t *stacks, int32_t *depths,
                                     void *cuda_stream)
{
    if (!target_tokens || !target_states || !target_stacks || !target_depths || !n_accepted ||
        !out_tokens || !states || !stacks || !depths || (k > 0 && !draft_tokens))
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_accept_draft: null pointer");
    if (k < 0 || batch < 0 || stack_cap < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_pda_accept_draft: k = %d, batch = %d, stack_cap = %d",
                         k, batch, stack_cap);
    if (batch == 0)
        return CSTR_OK;
    pda_accept_draft_kernel<<<(batch + 127) / 128, 128, 0, (cudaStream_t)cuda_stream>>>(
        draft_tokens, target_tokens, target_states, target_stacks, target_depths, k, batch,
        stack_cap, n_accepted, out_tokens, states, stacks, depths);
    CSTR_CUDA_TRY(cudaGetLastError());
    return CSTR_OK;
}

extern "C" int cstr_pda_step_status(cstr_pda_workspace_t *ws, void *cuda_stream, int64_t *bad_rows,
                                    int64_t *empty_mask_rows, int64_t *overflow_rows)
{
    if (!ws)
        return cstr_fail(CSTR_ERR_NULL, "cstr_pda_step_status: null workspace");
    int rc = cstr_check_device(ws->device, "PDA workspace");
    if (rc)
        return rc;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long host[3] = {0, 0, 0};
    CSTR_CUDA_TRY(cudaMemcpyAsync(host, ws->counters + 2, 24, cudaMemcpyDeviceToHost, stream));
    CSTR_CUDA_TRY(cudaMemsetAsync(ws->counters + 2, 0, 24, stream));
    CSTR_CUDA_TRY(cudaStreamSynchronize(stream));
    if (bad_rows)
        *bad_rows = (int64_t)host[0];
    if (empty_mask_rows)
        *empty_mask_rows = (int64_t)host[1];
    if (overflow_rows)
        *overflow_rows = (int64_t)host[2];
    return CSTR_OK;
}
