// Token-table builder: next[q][v] = delta*(q, bytes(v)) and the allowed-token
// bitmask, for every DFA state q and vocabulary token v (Algorithm 1 composed
// with the DFA as in Algorithm 2; Theorem 2 fixes the meaning).
//
// Work decomposition: a CTA owns 256 consecutive tokens (one per thread, the
// first 16 bytes of the token held in four registers) and a block of
// consecutive states; for each state every lane walks its own token through
// the DFA, the warp votes the 32 results into one mask word with a ballot, and
// the next-state entries go out as one coalesced row segment.  The DFA is read
// through the read-only path (it stays resident in L1/L2: 512 bytes per state
// as int16).
#include "cstr_internal.cuh"

namespace {

constexpr int kBuildThreads = 256;

template <typename DT, typename NT>
__global__ void __launch_bounds__(kBuildThreads)
build_rows_kernel(const DT *__restrict__ dfa, int n_states, const uint8_t *__restrict__ accept,
                  const uint4 *__restrict__ head, const uint32_t *__restrict__ len_arr,
                  const uint8_t *__restrict__ bytes, const uint32_t *__restrict__ off, int V,
                  int eos_id, NT *__restrict__ next, int64_t ldn, uint32_t *__restrict__ mask,
                  int64_t ldw, int states_per_cta)
{
    const int v = blockIdx.x * kBuildThreads + threadIdx.x;
    const bool in_vocab = v < V;
    uint4 rec = make_uint4(0, 0, 0, 0);
    uint32_t len = 0;
    uint32_t begin = 0;
    if (in_vocab) {
        rec = head[v];
        len = len_arr[v];
        begin = off[v];
    }
    const uint32_t w[4] = {rec.x, rec.y, rec.z, rec.w};
    const int q0 = blockIdx.y * states_per_cta;
    const int q1 = min(n_states, q0 + states_per_cta);
    const bool is_eos = in_vocab && v == eos_id;

    for (int q = q0; q < q1; ++q) {
        int s = (len > 0) ? q : CSTR_DEAD;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const bool go = (k < (int)len) && (s >= 0);
            if (!__any_sync(0xffffffffu, go))
                break;
            if (go) {
                const uint32_t b = (w[k >> 2] >> (8 * (k & 3))) & 0xffu;
                s = (int)__ldg(dfa + (int64_t)s * 256 + b);
            }
        }
        if (len > 16 && s >= 0) {       // rare: tokens longer than the packed head
            for (uint32_t k = 16; k < len; ++k) {
                s = (int)__ldg(dfa + (int64_t)s * 256 + bytes[begin + k]);
                if (s < 0)
                    break;
            }
        }
        bool allowed = s >= 0;
        if (is_eos) {                   // allowed exactly in accepting states; finishes the row
            allowed = accept[q] != 0;
            s = CSTR_DEAD;
        }
        const uint32_t word = __ballot_sync(0xffffffffu, allowed && in_vocab);
        if (in_vocab)
            next[(int64_t)q * ldn + v] = (NT)s;
        if ((threadIdx.x & 31) == 0 && in_vocab)
            mask[(int64_t)q * ldw + (v >> 5)] = word;
    }
}

}  // namespace

int cstr_launch_build(cstr_table *t, const cstr_dfa *dfa, cudaStream_t stream)
{
    const cstr_vocab *vc = t->vocab;
    const int states_per_cta = 16;
    dim3 grid((unsigned)((t->V + kBuildThreads - 1) / kBuildThreads),
              (unsigned)((dfa->n_states + states_per_cta - 1) / states_per_cta));
    if (grid.y > 65535u)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_table_build: %d states exceed the launch limit",
                         dfa->n_states);
    // The DFA's entry width follows its own size, the table's its capacity.
#define CSTR_BUILD(DT, NT)                                                                   \
    build_rows_kernel<DT, NT><<<grid, kBuildThreads, 0, stream>>>(                           \
        (const DT *)dfa->trans, dfa->n_states, dfa->accept, vc->head, vc->len, vc->bytes,    \
        vc->off, t->V, t->eos_id, (NT *)t->next, t->ldn, t->mask, t->ldw, states_per_cta)
    if (!dfa->wide && !t->wide)
        CSTR_BUILD(int16_t, int16_t);
    else if (!dfa->wide && t->wide)
        CSTR_BUILD(int16_t, int32_t);
    else if (dfa->wide && t->wide)
        CSTR_BUILD(int32_t, int32_t);
    else
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_table_build: DFA wider than the table");
#undef CSTR_BUILD
    CSTR_CUDA_TRY(cudaGetLastError());
    return CSTR_OK;
}
