// libcstr host side: handles, validation, uploads, table download, errors.
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <vector>

#include "cstr_internal.cuh"

static thread_local char g_err[512] = "";

int cstr_fail(int code, const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
    return code;
}

extern "C" const char *cstr_last_error(void) { return g_err; }

int cstr_check_device(int handle_device, const char *what)
{
    int cur = -1;
    CSTR_CUDA_TRY(cudaGetDevice(&cur));
    if (cur != handle_device)
        return cstr_fail(CSTR_ERR_DEVICE, "%s was created on device %d but device %d is current",
                         what, handle_device, cur);
    return CSTR_OK;
}

// --------------------------------------------- checking build: bounds record

#ifdef CSTR_BOUNDS_CHECK
#include <mutex>
#include "cstr_debug.h"

namespace {
std::mutex g_oob_mutex;
unsigned long long *g_oob_ptr[64] = {nullptr};
}  // namespace

unsigned long long *cstr_oob_record()
{
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64)
        return nullptr;
    std::lock_guard<std::mutex> lock(g_oob_mutex);
    if (!g_oob_ptr[device]) {
        unsigned long long *ptr = nullptr;
        if (cudaMalloc((void **)&ptr, 32) != cudaSuccess || cudaMemset(ptr, 0, 32) != cudaSuccess)
            return nullptr;
        g_oob_ptr[device] = ptr;
    }
    return g_oob_ptr[device];
}

extern "C" int cstr_debug_bounds_status(uint64_t *out, int32_t reset)
{
    if (!out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_debug_bounds_status: null pointer");
    unsigned long long *rec = cstr_oob_record();
    if (!rec)
        return cstr_fail(CSTR_ERR_CUDA, "cstr_debug_bounds_status: no record on this device");
    CSTR_CUDA_TRY(cudaDeviceSynchronize());
    unsigned long long host[4];
    CSTR_CUDA_TRY(cudaMemcpy(host, rec, 32, cudaMemcpyDeviceToHost));
    for (int i = 0; i < 4; ++i)
        out[i] = host[i];
    if (reset)
        CSTR_CUDA_TRY(cudaMemset(rec, 0, 32));
    return CSTR_OK;
}
#endif

// ------------------------------------------------------------------ DFA

namespace {

// Two order-independent 64-bit hashes per byte column of the raw table
// (thread = byte, a block sums a slab of rows, slabs combine with atomicAdd);
// the same pass checks that every target is a state or -1 and counts the
// bytes that have an edge out of each state.
__global__ void __launch_bounds__(256)
dfa_column_hash_kernel(const int32_t *__restrict__ raw, int n_states, int rows_per_block,
                       unsigned long long *__restrict__ hashes, uint16_t *__restrict__ degree)
{
    const int b = threadIdx.x;
    const int q0 = blockIdx.x * rows_per_block;
    const int q1 = min(n_states, q0 + rows_per_block);
    unsigned long long h1 = 0, h2 = 0;
    bool invalid = false;                    // a target outside [-1, n_states): hashes[513] != 0
    for (int q = q0; q < q1; ++q) {
        const int32_t target = raw[(long long)q * 256 + b];
        invalid |= target < -1 || target >= n_states;
        const int edges = __syncthreads_count(target >= 0);      // bytes with an edge out of q
        if (b == 0)
            degree[q] = (uint16_t)edges;
        unsigned long long x = (unsigned long long)(unsigned)target +
                               ((unsigned long long)(unsigned)q << 32) + 0x9e3779b97f4a7c15ull;
        x ^= x >> 30; x *= 0xbf58476d1ce4e5b9ull;        // splitmix64 finaliser: (q, value) -> 64 bits
        x ^= x >> 27; x *= 0x94d049bb133111ebull;
        x ^= x >> 31;
        h1 += x;
        h2 += (x ^ 0xc2b2ae3d27d4eb4full) * 0xff51afd7ed558ccdull;
    }
    atomicAdd(hashes + b, h1);
    atomicAdd(hashes + 256 + b, h2);
    if (invalid)
        atomicOr(hashes + 513, 1ull);
}

// Class-major code table from the raw table, proving the proposed classes on
// the way: tt[c][PERM(q)] = code(raw[q][rep[c]] or sink), q and the targets
// taken through `rank` when the automaton is renumbered; every raw[q][b] must
// equal raw[q][rep[cls[b]]], else *mismatch is set.  A block handles 8 states.
__global__ void __launch_bounds__(256)
dfa_build_table_kernel(const int32_t *__restrict__ raw, int n_states, int row, int n_classes,
                       const uint8_t *__restrict__ cls, const uint8_t *__restrict__ rep, int wide,
                       const int32_t *__restrict__ rank, void *__restrict__ tt,
                       unsigned long long *__restrict__ mismatch)
{
    __shared__ int32_t s_row[8][256];
    const int b = threadIdx.x;
    const int q0 = blockIdx.x * 8;
    bool differs = false;
    for (int i = 0; i < 8; ++i) {
        const int q = q0 + i;
        s_row[i][b] = (q < n_states) ? raw[(long long)q * 256 + b] : -1;
    }
    __syncthreads();
    const int my_rep = rep[cls[b]];
    for (int i = 0; i < 8; ++i)
        differs |= s_row[i][b] != s_row[i][my_rep];
    if (differs)
        atomicOr(mismatch, 1ull);
    for (int k = threadIdx.x; k < 8 * n_classes; k += 256) {
        const int i = k & 7, c = k >> 3;
        const int q = q0 + i;
        if (q >= row)
            continue;
        // slots and targets in internal ids (the sink and the padding slots map to themselves)
        const int32_t t = s_row[i][rep[c]];
        const int ti = t >= 0 ? (rank ? rank[t] : t) : n_states;
        const int qi = (rank && q < n_states) ? rank[q] : q;
        const unsigned target = (unsigned)CSTR_PERM(ti);
        const long long at = (long long)c * row + CSTR_PERM(qi);
        if (wide)
            ((uint32_t *)tt)[at] = target * 4u;
        else
            ((uint16_t *)tt)[at] = (uint16_t)(target * 2u);
    }
}

}  // namespace


// Host scan for the first target outside [-1, n_states): sets the error text and
// returns CSTR_ERR_DFA, or 0 if the table is well formed.
static int first_bad_target(const int32_t *trans, int32_t n_states)
{
    const int64_t n = (int64_t)n_states * 256;
    int bad = 0;                   // branch-free so that the scan vectorises
    for (int64_t i = 0; i < n; ++i)
        bad |= (trans[i] < -1) | (trans[i] >= n_states);
    if (!bad)
        return 0;
    for (int64_t i = 0; i < n; ++i) {
        if (trans[i] < -1 || trans[i] >= n_states)
            return cstr_fail(CSTR_ERR_DFA,
                             "cstr_load_dfa: state %lld byte %lld has target %d outside [-1, %d)",
                             (long long)(i / 256), (long long)(i % 256), trans[i], n_states);
    }
    return 0;
}

// Device scratch of cstr_load_dfa (the raw table and a few flags).  Allocating
// and freeing it cost more than the load's kernels, so each host thread keeps
// one block per process (at most kScratchKeep bytes, on the device it was last
// used on); larger requests are allocated and freed per call.
namespace {
constexpr int32_t kHostPathStates = 512;   // cstr_load_dfa: at or below, no device pre-processing
constexpr int kManyBytes = 64;             // a state with edges on this many bytes "allows many"
constexpr size_t kScratchKeep = 64u << 20;
struct ScratchCache {
    int device = -1;
    unsigned char *ptr = nullptr;
    size_t bytes = 0;
    // A host thread that ends gives its block back (a pool that recycles threads
    // would otherwise leak one block per dead thread).  At process exit the CUDA
    // runtime may already be gone; the calls then fail harmlessly.
    ~ScratchCache()
    {
        if (!ptr)
            return;
        int cur = -1;
        if (cudaGetDevice(&cur) != cudaSuccess)
            return;
        if (cur != device && cudaSetDevice(device) != cudaSuccess)
            return;
        cudaFree(ptr);
        if (cur != device)
            cudaSetDevice(cur);
        ptr = nullptr;
    }
};
thread_local ScratchCache t_scratch;

cudaError_t scratch_acquire(int device, size_t bytes, unsigned char **out, bool *cached)
{
    *cached = false;
    if (bytes > kScratchKeep)
        return cudaMalloc((void **)out, bytes);
    ScratchCache &c = t_scratch;
    if (c.ptr && (c.device != device || c.bytes < bytes)) {
        int cur = -1;                            // free on the device that owns the block
        cudaGetDevice(&cur);
        cudaSetDevice(c.device);
        cudaFree(c.ptr);
        cudaSetDevice(cur);
        c.ptr = nullptr;
        c.bytes = 0;
    }
    if (!c.ptr) {
        cudaError_t e = cudaMalloc((void **)&c.ptr, bytes);
        if (e != cudaSuccess) {
            c.ptr = nullptr;
            return e;
        }
        c.device = device;
        c.bytes = bytes;
    }
    *out = c.ptr;
    *cached = true;
    return cudaSuccess;
}

void scratch_release(unsigned char *ptr, bool cached)
{
    if (!cached)
        cudaFree(ptr);
}
}  // namespace

extern "C" void cstr_free_dfa(cstr_dfa_t *dfa)
{
    if (!dfa)
        return;
    cudaFree(dfa->tt);
    cudaFree(dfa->cls);                  // one allocation: byte classes, then the accept flags
    cudaFree(dfa->tstate);
    cudaFree(dfa->tset);
    cudaFree(dfa->ttarget);
    cudaFree(dfa->rank);                 // one allocation: rank, then unrank
    free(dfa->rank_host);
    delete dfa;
}

extern "C" int cstr_load_dfa(const int32_t *trans, const uint8_t *accept, int32_t n_states,
                             int32_t start_state, cstr_dfa_t **out)
{
    if (!trans || !accept || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_dfa: null pointer");
    *out = nullptr;
    if (n_states < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_dfa: n_states = %d, need >= 1", n_states);
    if (n_states > 4000000)       // row byte offsets of the class-major table are 32-bit
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_dfa: n_states = %d, at most 4,000,000 supported",
                         n_states);
    if (start_state < 0 || start_state >= n_states)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_dfa: start_state %d outside [0, %d)",
                         start_state, n_states);
    const int64_t n = (int64_t)n_states * 256;
    cstr_dfa *d = new (std::nothrow) cstr_dfa();
    if (!d)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa: out of host memory");
    memset(d, 0, sizeof *d);
    d->n_states = n_states;
    d->start = start_state;
    d->wide = (int64_t)n_states + 1 > 32767;
    d->row = ((int64_t)n_states + 1 + 255) / 256 * 256;
    const size_t esz = d->wide ? 4 : 2;

    // The raw table goes to the device once; validation, byte classes (bytes whose
    // columns are identical in every state) and the class-major code table are
    // made there: one pass checks the targets and hashes the columns, the hashes
    // propose the classes, a second kernel proves them entry by entry while it
    // writes the table, and only a hash collision (never seen) falls back to
    // exact column comparisons on the host.
    std::vector<uint8_t> flags;
    try {
        flags.resize(n_states);
    } catch (const std::bad_alloc &) {
        delete d;
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa: out of host memory");
    }
    for (int32_t q = 0; q < n_states; ++q)
        flags[q] = accept[q] ? 1 : 0;

    // Small automata: everything on the host (the table is a few hundred KB at
    // most), two allocations and two uploads instead of a dozen driver calls.
    if (n_states <= kHostPathStates) {
        int rc = first_bad_target(trans, n_states);
        if (rc) {
            delete d;
            return rc;
        }
        uint8_t cls_h[256], rep_h[256];
        int nc = 0;
        for (int b = 0; b < 256; ++b) {              // classes numbered by their smallest byte
            int found = -1;
            for (int c = 0; c < nc && found < 0; ++c) {
                bool same = true;
                for (int32_t q = 0; q < n_states && same; ++q)
                    same = trans[(size_t)q * 256 + b] == trans[(size_t)q * 256 + rep_h[c]];
                if (same)
                    found = c;
            }
            if (found < 0) {
                found = nc;
                rep_h[nc++] = (uint8_t)b;
            }
            cls_h[b] = (uint8_t)found;
        }
        d->n_classes = nc;
        std::vector<uint16_t> tt_h;                  // n_states <= 32766 here: 16-bit entries
        std::vector<uint8_t> small_h;
        try {
            tt_h.resize((size_t)nc * (size_t)d->row);
            small_h.resize(256 + (size_t)n_states);
        } catch (const std::bad_alloc &) {
            delete d;
            return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa: out of host memory");
        }
        for (int c = 0; c < nc; ++c)
            for (int64_t q = 0; q < d->row; ++q) {
                const int32_t t = q < n_states ? trans[(size_t)q * 256 + rep_h[c]] : -1;
                tt_h[(size_t)c * d->row + CSTR_PERM(q)] =
                    (uint16_t)(CSTR_PERM(t >= 0 ? t : n_states) * 2);
            }
        memcpy(small_h.data(), cls_h, 256);
        memcpy(small_h.data() + 256, flags.data(), (size_t)n_states);
        cudaError_t e = cudaGetDevice(&d->device);
        if (e == cudaSuccess)
            e = cudaMalloc((void **)&d->cls, small_h.size());
        d->accept = d->cls ? d->cls + 256 : nullptr;
        if (e == cudaSuccess)
            e = cudaMalloc(&d->tt, tt_h.size() * 2);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->cls, small_h.data(), small_h.size(), cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->tt, tt_h.data(), tt_h.size() * 2, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                           "cstr_load_dfa: %s", cudaGetErrorString(e));
            cstr_free_dfa(d);
            return rc;
        }
        *out = d;
        return CSTR_OK;
    }

    // temporaries in one block: [raw table][2 x 256 hashes, mismatch flag, invalid flag][256 reps]
    const size_t raw_bytes = (size_t)n * 4, hash_bytes = 514 * 8;
    cudaError_t e = cudaGetDevice(&d->device);
    unsigned char *temp = nullptr;
    bool temp_cached = false;
    if (e == cudaSuccess)
        e = scratch_acquire(d->device, raw_bytes + hash_bytes + 256 + (size_t)n_states * 2, &temp,
                            &temp_cached);
    if (e != cudaSuccess) {
        // No usable device: still tell the caller about a malformed table first.
        const int rc_dfa = first_bad_target(trans, n_states);
        const int rc = rc_dfa ? rc_dfa
                              : cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                                          "cstr_load_dfa: %s", cudaGetErrorString(e));
        delete d;
        return rc;
    }
    int32_t *raw = (int32_t *)temp;
    unsigned long long *hashes = (unsigned long long *)(temp + raw_bytes);
    uint8_t *rep_dev = temp + raw_bytes + hash_bytes;
    uint16_t *degree_dev = (uint16_t *)(temp + raw_bytes + hash_bytes + 256);
    e = cudaMalloc((void **)&d->cls, 256 + (size_t)n_states);
    d->accept = d->cls ? d->cls + 256 : nullptr;
    if (e == cudaSuccess)
        e = cudaMemcpy(raw, trans, raw_bytes, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(d->accept, flags.data(), (size_t)n_states, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemset(hashes, 0, hash_bytes);
    unsigned long long host_hash[514];
    if (e == cudaSuccess) {
        const int rows_per_block = 64;
        dfa_column_hash_kernel<<<(n_states + rows_per_block - 1) / rows_per_block, 256>>>(
            raw, n_states, rows_per_block, hashes, degree_dev);
        e = cudaGetLastError();
    }
    std::vector<uint16_t> degree;
    if (e == cudaSuccess) {
        try {
            degree.resize((size_t)n_states);
        } catch (const std::bad_alloc &) {
            scratch_release(temp, temp_cached);
            cstr_free_dfa(d);
            return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa: out of host memory");
        }
        e = cudaMemcpy(host_hash, hashes, hash_bytes, cudaMemcpyDeviceToHost);
    }
    if (e == cudaSuccess)
        e = cudaMemcpy(degree.data(), degree_dev, (size_t)n_states * 2, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && host_hash[513] != 0) {       // some target is out of range: say which
        scratch_release(temp, temp_cached);
        cstr_free_dfa(d);
        const int rc = first_bad_target(trans, n_states);
        return rc ? rc : cstr_fail(CSTR_ERR_DFA, "cstr_load_dfa: a target is outside [-1, %d)",
                                   n_states);
    }

    // Sparse automata: when at least one warp's worth of states (256) allows few
    // bytes each, the builder prunes per warp, and the states that allow many
    // bytes are numbered first so that they do not keep every warp alive.
    if (e == cudaSuccess && host_hash[513] == 0) {
        int32_t many = 0;
        for (int32_t q = 0; q < n_states; ++q)
            many += degree[q] >= kManyBytes;
        d->sparse = n_states - many >= 256;
        d->n_many = many;
        bool in_order = true;                    // already "many first"?
        for (int32_t q = 0; q + 1 < n_states && in_order; ++q)
            in_order = !(degree[q] < kManyBytes && degree[q + 1] >= kManyBytes);
        if (d->sparse && many > 0 && !in_order) {
            d->rank_host = (int32_t *)malloc(((size_t)n_states + 1) * 4);
            std::vector<int32_t> unrank;
            try {
                unrank.resize((size_t)n_states + 1);
            } catch (const std::bad_alloc &) {
                free(d->rank_host);
                d->rank_host = nullptr;
            }
            if (!d->rank_host) {
                scratch_release(temp, temp_cached);
                cstr_free_dfa(d);
                return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa: out of host memory");
            }
            int32_t at_many = 0, at_few = many;  // stable: each group keeps the caller's order
            for (int32_t q = 0; q < n_states; ++q) {
                const int32_t r = degree[q] >= kManyBytes ? at_many++ : at_few++;
                d->rank_host[q] = r;
                unrank[r] = q;
            }
            d->rank_host[n_states] = n_states;
            unrank[n_states] = n_states;
            e = cudaMalloc((void **)&d->rank, ((size_t)n_states + 1) * 8);   // rank, then unrank
            d->unrank = d->rank ? d->rank + n_states + 1 : nullptr;
            if (e == cudaSuccess)
                e = cudaMemcpy(d->rank, d->rank_host, ((size_t)n_states + 1) * 4,
                               cudaMemcpyHostToDevice);
            if (e == cudaSuccess)
                e = cudaMemcpy(d->unrank, unrank.data(), ((size_t)n_states + 1) * 4,
                               cudaMemcpyHostToDevice);
        }
    }

    uint8_t cls8[256], rep8[256];
    int n_classes = 0;
    auto propose = [&](bool exact) {
        n_classes = 0;
        for (int b = 0; b < 256; ++b) {
            int found = -1;
            for (int c = 0; c < n_classes && found < 0; ++c) {
                const int r = rep8[c];
                bool same = host_hash[b] == host_hash[r] && host_hash[256 + b] == host_hash[256 + r];
                if (exact) {
                    same = true;
                    for (int32_t q = 0; q < n_states && same; ++q)
                        same = trans[(size_t)q * 256 + b] == trans[(size_t)q * 256 + r];
                }
                if (same)
                    found = c;
            }
            if (found < 0) {                     // classes are numbered by their smallest byte
                found = n_classes;
                rep8[n_classes++] = (uint8_t)b;
            }
            cls8[b] = (uint8_t)found;
        }
    };
    for (int attempt = 0; attempt < 2 && e == cudaSuccess; ++attempt) {
        propose(attempt == 1);
        d->n_classes = n_classes;
        const size_t tt_bytes = (size_t)n_classes * (size_t)d->row * esz;
        cudaFree(d->tt);
        d->tt = nullptr;
        e = cudaMalloc(&d->tt, tt_bytes);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->cls, cls8, 256, cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(rep_dev, rep8, 256, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) {
            dfa_build_table_kernel<<<(unsigned)((d->row + 7) / 8), 256>>>(
                raw, n_states, (int)d->row, n_classes, d->cls, rep_dev, d->wide, d->rank, d->tt,
                hashes + 512);
            e = cudaGetLastError();
        }
        unsigned long long mismatch = 0;
        if (e == cudaSuccess)
            e = cudaMemcpy(&mismatch, hashes + 512, 8, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess || mismatch == 0)
            break;                               // proven (or failed): no second attempt
        e = cudaMemset(hashes + 512, 0, 8);      // a collision: redo with exact classes
    }
    scratch_release(temp, temp_cached);
    if (e != cudaSuccess) {
        int rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                           "cstr_load_dfa: %s", cudaGetErrorString(e));
        cstr_free_dfa(d);
        return rc;
    }
    *out = d;
    return CSTR_OK;
}

extern "C" int cstr_load_dfa_terminals(const int32_t *trans, const int32_t *term_trans,
                                       int32_t n_labels, const uint8_t *accept, int32_t n_states,
                                       int32_t start_state, cstr_dfa_t **out)
{
    if (!out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_dfa_terminals: null pointer");
    *out = nullptr;
    if (n_labels < 0 || n_labels > 32)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_dfa_terminals: n_labels = %d, need 0..32",
                         n_labels);
    if (n_labels > 0 && !term_trans)
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_dfa_terminals: null term_trans");
    if (n_states >= 1) {
        for (int64_t i = 0; i < (int64_t)n_states * n_labels; ++i) {
            if (term_trans[i] < -1 || term_trans[i] >= n_states)
                return cstr_fail(CSTR_ERR_DFA,
                                 "cstr_load_dfa_terminals: state %lld label %lld has target %d "
                                 "outside [-1, %d)", (long long)(i / n_labels),
                                 (long long)(i % n_labels), term_trans[i], n_states);
        }
    }
    cstr_dfa *d = nullptr;
    int rc = cstr_load_dfa(trans, accept, n_states, start_state, &d);
    if (rc)
        return rc;
    d->n_labels = n_labels;
    std::vector<int32_t> tstate;
    std::vector<uint32_t> tset, ttarget;
    try {
        for (int32_t q = 0; q < n_states && n_labels > 0; ++q) {
            uint32_t labels = 0;
            for (int32_t t = 0; t < n_labels; ++t)
                if (term_trans[(int64_t)q * n_labels + t] >= 0)
                    labels |= 1u << t;
            if (!labels)
                continue;
            tstate.push_back(q);
            tset.push_back(labels);
            for (int32_t t = 0; t < n_labels; ++t) {
                int32_t target = term_trans[(int64_t)q * n_labels + t];
                if (target >= 0 && d->rank_host)         // table entries hold internal ids
                    target = d->rank_host[target];
                const uint32_t code = (uint32_t)CSTR_PERM(target < 0 ? n_states : target)
                                      << (d->wide ? 2 : 1);
                ttarget.push_back(code);
            }
        }
    } catch (const std::bad_alloc &) {
        cstr_free_dfa(d);
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_dfa_terminals: out of host memory");
    }
    d->n_term_states = (int32_t)tstate.size();
    if (d->n_term_states > 0) {
        cudaError_t e = cudaMalloc((void **)&d->tstate, tstate.size() * 4);
        if (e == cudaSuccess)
            e = cudaMalloc((void **)&d->tset, tset.size() * 4);
        if (e == cudaSuccess)
            e = cudaMalloc((void **)&d->ttarget, ttarget.size() * 4);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->tstate, tstate.data(), tstate.size() * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->tset, tset.data(), tset.size() * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess)
            e = cudaMemcpy(d->ttarget, ttarget.data(), ttarget.size() * 4, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                           "cstr_load_dfa_terminals: %s", cudaGetErrorString(e));
            cstr_free_dfa(d);
            return rc;
        }
    }
    *out = d;
    return CSTR_OK;
}

// ---------------------------------------------------------------- vocab

extern "C" int cstr_vocab_set_token_sets(cstr_vocab_t *vocab, const uint32_t *token_sets,
                                         int32_t n_labels)
{
    if (!vocab || !token_sets)
        return cstr_fail(CSTR_ERR_NULL, "cstr_vocab_set_token_sets: null pointer");
    if (n_labels < 1 || n_labels > 32)
        return cstr_fail(CSTR_ERR_ARG, "cstr_vocab_set_token_sets: n_labels = %d, need 1..32",
                         n_labels);
    int rc = cstr_check_device(vocab->device, "vocabulary");
    if (rc)
        return rc;
    uint32_t *dev = nullptr;
    CSTR_CUDA_TRY(cudaMalloc((void **)&dev, (size_t)vocab->V * 4));
    cudaError_t e = cudaMemcpy(dev, token_sets, (size_t)vocab->V * 4, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(dev);
        return cstr_fail(CSTR_ERR_CUDA, "cstr_vocab_set_token_sets: %s", cudaGetErrorString(e));
    }
    cudaFree(vocab->tsets);
    vocab->tsets = dev;
    vocab->n_labels = n_labels;
    return CSTR_OK;
}

extern "C" void cstr_free_vocab(cstr_vocab_t *v)
{
    if (!v)
        return;
    cudaFree(v->bytes);
    cudaFree(v->off);
    cudaFree(v->desc);
    cudaFree(v->pre4);
    cudaFree(v->by_len);
    cudaFree(v->tsets);
    delete v;
}

extern "C" int cstr_load_vocab(const uint8_t *vocab_bytes, const int64_t *offsets,
                               int32_t vocab_size, cstr_vocab_t **out)
{
    if (!offsets || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_vocab: null pointer");
    *out = nullptr;
    if (vocab_size < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_load_vocab: vocab_size = %d, need >= 1", vocab_size);
    if (offsets[0] != 0)
        return cstr_fail(CSTR_ERR_VOCAB, "cstr_load_vocab: offsets[0] = %lld, need 0",
                         (long long)offsets[0]);
    for (int32_t v = 0; v < vocab_size; ++v) {
        if (offsets[v + 1] < offsets[v])
            return cstr_fail(CSTR_ERR_VOCAB, "cstr_load_vocab: offsets decrease at token %d", v);
        if (offsets[v + 1] - offsets[v] >= (1 << 24))
            return cstr_fail(CSTR_ERR_VOCAB, "cstr_load_vocab: token %d is longer than 2^24 bytes",
                             v);
    }
    const int64_t total = offsets[vocab_size];
    if (total >= ((int64_t)1 << 31))
        return cstr_fail(CSTR_ERR_VOCAB, "cstr_load_vocab: %lld vocabulary bytes, need < 2^31",
                         (long long)total);
    if (total > 0 && !vocab_bytes)
        return cstr_fail(CSTR_ERR_NULL, "cstr_load_vocab: null vocab_bytes");

    cstr_vocab *vh = new (std::nothrow) cstr_vocab();
    if (!vh)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_vocab: out of host memory");
    memset(vh, 0, sizeof *vh);
    vh->V = vocab_size;
    vh->total_bytes = total;

    std::vector<uint32_t> off32;
    std::vector<int32_t> order;
    std::vector<uint4> desc;
    std::vector<uint32_t> pre4;
    uint32_t max_len = 0;
    try {
        off32.resize((size_t)vocab_size + 1);
        order.resize((size_t)vocab_size);
        desc.resize((size_t)vocab_size);
        pre4.resize((size_t)vocab_size);
        for (int32_t v = 0; v <= vocab_size; ++v)
            off32[v] = (uint32_t)offsets[v];
        // lexicographic order of the byte strings (a prefix sorts before its
        // extensions), ties by id: the depth-first order of the vocabulary trie.
        // Sort keys carry the first 8 bytes as a big-endian integer, so that most
        // comparisons never touch the strings.
        struct SortKey {
            uint64_t head;
            uint32_t len;
            int32_t id;
        };
        std::vector<SortKey> keys((size_t)vocab_size);
        for (int32_t v = 0; v < vocab_size; ++v) {
            const uint32_t len = off32[v + 1] - off32[v];
            uint64_t head = 0;
            for (uint32_t k = 0; k < 8; ++k)
                head = (head << 8) | (k < len ? (uint64_t)vocab_bytes[off32[v] + k] : 0u);
            keys[v].head = head;
            keys[v].len = len;
            keys[v].id = v;
        }
        auto full_less = [&](const SortKey &x, const SortKey &y) {
            if (x.head != y.head)
                return x.head < y.head;
            const int32_t a = x.id, b = y.id;
            const uint32_t la = x.len, lb = y.len;
            if (la > 8 && lb > 8) {              // equal first 8 bytes: compare the rest
                const uint32_t m = (la < lb ? la : lb) - 8;
                const int c = memcmp(vocab_bytes + off32[a] + 8, vocab_bytes + off32[b] + 8, m);
                if (c != 0)
                    return c < 0;
            }
            if (la != lb)
                return la < lb;
            return a < b;
        };
        // Stable radix passes, least significant digit first: min(length, 9), then
        // the head in four 16-bit digits.  Ids start in ascending order, so equal
        // (head, length <= 8) keys - equal strings - end up ordered by id, and a
        // token of at most 8 bytes precedes the longer ones it is a prefix of.
        // Runs of longer tokens with equal heads are finished by comparison.
        {
            std::vector<SortKey> tmp((size_t)vocab_size);
            std::vector<uint32_t> count(65536 + 1);
            SortKey *src = keys.data(), *dst = tmp.data();
            for (int pass = 0; pass < 5; ++pass) {
                auto digit = [pass](const SortKey &k) -> uint32_t {
                    if (pass == 0)
                        return k.len < 9 ? k.len : 9u;
                    return (uint32_t)(k.head >> (16 * (pass - 1))) & 0xffffu;
                };
                std::fill(count.begin(), count.end(), 0u);
                for (int32_t i = 0; i < vocab_size; ++i)
                    ++count[digit(src[i]) + 1];
                for (uint32_t d = 0; d < 65536; ++d)
                    count[d + 1] += count[d];
                for (int32_t i = 0; i < vocab_size; ++i)
                    dst[count[digit(src[i])]++] = src[i];
                std::swap(src, dst);
            }
            if (src != keys.data())              // five passes: the result sits in tmp
                memcpy(keys.data(), src, (size_t)vocab_size * sizeof(SortKey));
        }
        for (int32_t i = 0; i < vocab_size;) {
            int32_t j = i + 1;
            if (keys[i].len > 8) {
                while (j < vocab_size && keys[j].head == keys[i].head && keys[j].len > 8)
                    ++j;
                if (j - i > 1)
                    std::sort(keys.begin() + i, keys.begin() + j, full_less);
            }
            i = j;
        }
        for (int32_t i = 0; i < vocab_size; ++i)
            order[i] = keys[i].id;
        for (int32_t i = 0; i < vocab_size; ++i) {
            const int32_t v = order[i];
            const uint8_t *cur = vocab_bytes + off32[v];
            const uint32_t n = off32[v + 1] - off32[v];
            if (n > max_len)
                max_len = n;
            uint32_t p = 0;
            if (i > 0) {
                const int32_t u = order[i - 1];
                const uint8_t *prev = vocab_bytes + off32[u];
                const uint32_t pn = off32[u + 1] - off32[u];
                const uint32_t m = n < pn ? n : pn;
                while (p < m && p < CSTR_STACK_DEPTH && prev[p] == cur[p])
                    ++p;
            }
            uint8_t sfx[8] = {0};
            for (uint32_t k = 0; k < 8 && p + k < n; ++k)
                sfx[k] = cur[p + k];
            uint4 r;
            r.x = (uint32_t)v;
            r.y = n | (p << 24);
            memcpy(&r.z, sfx, 4);
            memcpy(&r.w, sfx + 4, 4);
            desc[i] = r;
            uint32_t head = 0;                   // bytes 0..3: a walk that starts at this token
            for (uint32_t k = 0; k < 4 && k < n; ++k)    // needs them (its descriptor starts at p)
                head |= (uint32_t)cur[k] << (8 * k);
            pre4[i] = head;
        }
    } catch (const std::bad_alloc &) {
        delete vh;
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_vocab: out of host memory");
    }
    vh->max_len = max_len;
    // token ids by length (counting sort, stable in the id): a warp that takes 32
    // consecutive entries walks tokens of the same length
    std::vector<uint32_t> by_len;
    try {
        by_len.resize((size_t)vocab_size);
        std::vector<uint32_t> start(66, 0u);
        for (int32_t v = 0; v < vocab_size; ++v) {
            const uint32_t n = off32[v + 1] - off32[v];
            ++start[(n < 64 ? n : 64) + 1];
        }
        for (int k = 0; k < 65; ++k)
            start[k + 1] += start[k];
        for (int32_t v = 0; v < vocab_size; ++v) {
            const uint32_t n = off32[v + 1] - off32[v];
            by_len[start[n < 64 ? n : 64]++] = (uint32_t)v;
        }
    } catch (const std::bad_alloc &) {
        delete vh;
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_load_vocab: out of host memory");
    }

    cudaError_t e = cudaGetDevice(&vh->device);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&vh->bytes, (size_t)total + 16);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&vh->off, ((size_t)vocab_size + 1) * sizeof(uint32_t));
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&vh->desc, (size_t)vocab_size * sizeof(uint4));
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&vh->pre4, (size_t)vocab_size * sizeof(uint32_t));
    if (e == cudaSuccess)
        e = cudaMemcpy(vh->pre4, pre4.data(), pre4.size() * sizeof(uint32_t), cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&vh->by_len, (size_t)vocab_size * sizeof(uint32_t));
    if (e == cudaSuccess)
        e = cudaMemcpy(vh->by_len, by_len.data(), by_len.size() * sizeof(uint32_t),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemset(vh->bytes, 0, (size_t)total + 16);
    if (e == cudaSuccess && total > 0)
        e = cudaMemcpy(vh->bytes, vocab_bytes, (size_t)total, cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(vh->off, off32.data(), off32.size() * sizeof(uint32_t),
                       cudaMemcpyHostToDevice);
    if (e == cudaSuccess)
        e = cudaMemcpy(vh->desc, desc.data(), desc.size() * sizeof(uint4), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        int rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                           "cstr_load_vocab: %s", cudaGetErrorString(e));
        cstr_free_vocab(vh);
        return rc;
    }
    *out = vh;
    return CSTR_OK;
}

// ---------------------------------------------------------------- table

namespace {

// Logical view of a slab of states for cstr_table_download: out[q - q_lo][v] =
// state reached from q on token v, -1 for "no edge".  The device table is
// token-major (next[v][q]) and holds codes (CSTR_PERM(target) << shift, the sink
// n_states meaning "no edge"), so this is a decode plus a 32 x 32 tiled
// transpose through shared memory.  Block (32, 8); tile x = 32 tokens, y = 32
// states starting at a multiple of 32.
template <typename NT>
__global__ void __launch_bounds__(256)
table_decode_kernel(const NT *__restrict__ next, long long lds, int V, int q_lo, int rows,
                    int q_tile0, int n_states, int shift, const int32_t *__restrict__ rank,
                    const int32_t *__restrict__ unrank, int32_t *__restrict__ out,
                    unsigned long long *oob)
{
    __shared__ int32_t tile[32][33];
    const int v0 = blockIdx.x * 32;
    const int q0 = (q_tile0 + (int)blockIdx.y) * 32;
    const int tx = threadIdx.x, ty = threadIdx.y;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int v = v0 + ty + 8 * k, q = q0 + tx;
        int32_t u = -1;
        if (v < V && q < n_states) {                     // q < lds: inside the token's row
            const int qi = rank ? rank[q] : q;           // the table is indexed by internal ids
            const int32_t code = CSTR_INB(oob, qi, lds, CSTR_SITE_DOWNLOAD)
                                     ? (int32_t)next[(long long)v * lds + qi] : (n_states << shift);
            u = CSTR_UNPERM(code >> shift);
            if (u == n_states)
                u = -1;
            else if (unrank)
                u = unrank[u];
        }
        tile[ty + 8 * k][tx] = u;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int q = q0 + ty + 8 * k, v = v0 + tx;
        if (q >= q_lo && q < q_lo + rows && v < V &&
            CSTR_INB(oob, (long long)(q - q_lo) * V + v, (long long)rows * V, CSTR_SITE_DOWNLOAD))
            out[(long long)(q - q_lo) * V + v] = tile[tx][ty + 8 * k];
    }
}

}  // namespace

extern "C" void cstr_free_table(cstr_table_t *t)
{
    if (!t)
        return;
    cudaFree(t->next);
    cudaFree(t->mask);
    cudaFree(t->maskT);
    cudaFree(t->accept);
    cudaFree(t->group_key);
    cudaFree(t->group_min);
    cudaFree(t->group_rep);
    cudaFree(t->group_reptok);
    cudaFree(t->group_desc);
    cudaFree(t->group_count);
    cudaFree(t->group_uniq);
    cudaFree(t->group_blk);
    cudaFree(t->rank);                   // one allocation: rank, then unrank
    cudaFree(t->build_status);
    cstr_free_vocab(t->owned_vocab);
    delete t;
}

extern "C" int cstr_table_create(const cstr_vocab_t *vocab, int32_t max_states,
                                 cstr_table_t **out)
{
    if (!vocab || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_table_create: null pointer");
    *out = nullptr;
    if (max_states < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_table_create: max_states = %d, need >= 1", max_states);
    int rc = cstr_check_device(vocab->device, "vocabulary");
    if (rc)
        return rc;
    cstr_table *t = new (std::nothrow) cstr_table();
    if (!t)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_table_create: out of host memory");
    memset(t, 0, sizeof *t);
    t->device = vocab->device;
    t->vocab = vocab;
    t->max_states = max_states;
    t->V = vocab->V;
    t->W = (vocab->V + 31) / 32;
    t->lds = ((int64_t)max_states + 255) / 256 * 256;
    t->ldw = ((int64_t)t->W + 31) / 32 * 32;
    t->ldb = t->lds / 32 + 8 - (t->lds / 32) % 8;   // a multiple of 8, above lds / 32
    t->wide = (int64_t)max_states + 1 > 32767;
    t->eos_id = -1;
    const size_t next_bytes = (size_t)t->V * (size_t)t->lds * (t->wide ? 4 : 2);
    const size_t mask_bytes = (size_t)max_states * (size_t)t->ldw * 4;
    const size_t maskT_bytes = (size_t)t->V * (size_t)t->ldb * 4;
    cudaError_t e = cudaMalloc(&t->next, next_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->mask, mask_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->maskT, maskT_bytes);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->accept, (size_t)max_states);
    t->group_slots = 1024;
    while (t->group_slots < 4ull * (unsigned)t->V && t->group_slots < (1u << 30))
        t->group_slots <<= 1;
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_key, (size_t)t->group_slots * 8);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_min, (size_t)t->group_slots * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_rep, (size_t)t->V * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_reptok, (size_t)t->V * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_desc, (size_t)t->V * sizeof(uint4));
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_count, 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_uniq, (size_t)t->V * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->group_blk, ((size_t)t->V / 1024 + 1) * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->rank, ((size_t)max_states + 1) * 8);
    t->unrank = t->rank ? t->rank + max_states + 1 : nullptr;
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&t->build_status, 4);
    if (e == cudaSuccess)
        e = cudaMemset(t->build_status, 0, 4);
    if (e == cudaSuccess)
        e = cudaMemset(t->mask, 0, mask_bytes);   // padding words stay zero for good
    if (e == cudaSuccess)
        e = cudaMemset(t->accept, 0, (size_t)max_states);
    if (e != cudaSuccess) {
        rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                       "cstr_table_create (%zu + %zu bytes): %s", next_bytes, mask_bytes,
                       cudaGetErrorString(e));
        cstr_free_table(t);
        return rc;
    }
    *out = t;
    return CSTR_OK;
}

static int table_build_common(cstr_table_t *table, const cstr_dfa_t *dfa, int32_t eos_id,
                              void *cuda_stream, bool dense_walk)
{
    if (!table || !dfa)
        return cstr_fail(CSTR_ERR_NULL, "cstr_table_build: null pointer");
    int rc = cstr_check_device(table->device, "table");
    if (rc)
        return rc;
    if (dfa->device != table->device)
        return cstr_fail(CSTR_ERR_DEVICE, "cstr_table_build: DFA and table on different devices");
    if (dfa->n_states > table->max_states)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_table_build: DFA has %d states, table holds %d",
                         dfa->n_states, table->max_states);
    if (dfa->n_term_states > 0 && table->vocab->n_labels < dfa->n_labels)
        return cstr_fail(CSTR_ERR_SHAPE,
                         "cstr_table_build: the DFA uses %d terminal labels, the vocabulary has "
                         "token sets for %d (cstr_vocab_set_token_sets)", dfa->n_labels,
                         table->vocab->n_labels);
    if (eos_id < -1 || eos_id >= table->V)
        return cstr_fail(CSTR_ERR_ARG, "cstr_table_build: eos_id %d outside [-1, %d)", eos_id,
                         table->V);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    table->n_states = dfa->n_states;
    table->start = dfa->start;
    table->eos_id = eos_id;
    table->code_shift = dfa->wide ? 2 : 1;
    // the table keeps its own copy of the accept flags and of the state numbering; the builder
    // copies them on the device (cstr_launch_build)
    table->renumbered = dfa->rank != nullptr;
    table->unrank = table->rank + dfa->n_states + 1;     // as in the DFA: right behind rank
    return cstr_launch_build(table, dfa, stream, dense_walk);
}

extern "C" int cstr_table_build(cstr_table_t *table, const cstr_dfa_t *dfa, int32_t eos_id,
                                void *cuda_stream)
{
    return table_build_common(table, dfa, eos_id, cuda_stream, false);
}

extern "C" int cstr_table_build_dense(cstr_table_t *table, const cstr_dfa_t *dfa, int32_t eos_id,
                                      void *cuda_stream)
{
    return table_build_common(table, dfa, eos_id, cuda_stream, true);
}

extern "C" int cstr_build_token_table(const cstr_dfa_t *dfa, const uint8_t *vocab_bytes,
                                      const int64_t *offsets, int32_t vocab_size, int32_t eos_id,
                                      void *cuda_stream, cstr_table_t **out)
{
    if (!dfa || !out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_build_token_table: null pointer");
    *out = nullptr;
    cstr_vocab *vocab = nullptr;
    int rc = cstr_load_vocab(vocab_bytes, offsets, vocab_size, &vocab);
    if (rc)
        return rc;
    cstr_table *t = nullptr;
    rc = cstr_table_create(vocab, dfa->n_states, &t);
    if (rc) {
        cstr_free_vocab(vocab);
        return rc;
    }
    t->owned_vocab = vocab;
    rc = cstr_table_build(t, dfa, eos_id, cuda_stream);
    if (rc) {
        cstr_free_table(t);
        return rc;
    }
    *out = t;
    return CSTR_OK;
}

extern "C" int cstr_table_info(const cstr_table_t *t, int32_t *n_states, int32_t *vocab_size,
                               int32_t *mask_words, int32_t *start_state)
{
    if (!t)
        return cstr_fail(CSTR_ERR_NULL, "cstr_table_info: null table");
    if (n_states)
        *n_states = t->n_states;
    if (vocab_size)
        *vocab_size = t->V;
    if (mask_words)
        *mask_words = t->W;
    if (start_state)
        *start_state = t->start;
    return CSTR_OK;
}

extern "C" int cstr_table_download(const cstr_table_t *t, int32_t state_lo, int32_t state_hi,
                                   uint32_t *mask_host, int32_t *next_host, void *cuda_stream)
{
    if (!t)
        return cstr_fail(CSTR_ERR_NULL, "cstr_table_download: null table");
    int rc = cstr_check_device(t->device, "table");
    if (rc)
        return rc;
    if (state_lo < 0 || state_hi < state_lo || state_hi > t->n_states)
        return cstr_fail(CSTR_ERR_ARG, "cstr_table_download: states [%d, %d) outside [0, %d)",
                         state_lo, state_hi, t->n_states);
    CSTR_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    unsigned int build_status = 0;
    CSTR_CUDA_TRY(cudaMemcpy(&build_status, t->build_status, 4, cudaMemcpyDeviceToHost));
    if (build_status != 0)
        return cstr_fail(CSTR_ERR_CUDA, "cstr_table_download: a build of this table gave up waiting "
                         "for its staged rows (status %u); the table is incomplete", build_status);
    const int32_t rows = state_hi - state_lo;
    if (rows == 0)
        return CSTR_OK;
    if (mask_host) {
        CSTR_CUDA_TRY(cudaMemcpy2D(mask_host, (size_t)t->W * 4, t->mask + (int64_t)state_lo * t->ldw,
                                   (size_t)t->ldw * 4, (size_t)t->W * 4, rows,
                                   cudaMemcpyDeviceToHost));
    }
    if (next_host) {
        // The device table is token-major and holds codes; a kernel decodes and
        // transposes a slab of states into the logical layout, which then comes
        // down as one contiguous copy per slab.
        const int64_t slab_bytes_max = 256ll << 20;
        int64_t slab = slab_bytes_max / ((int64_t)t->V * 4);
        slab = slab < 32 ? 32 : slab / 32 * 32;
        if (slab > rows)
            slab = rows;
        int32_t *stage = nullptr;
        CSTR_CUDA_TRY(cudaMalloc((void **)&stage, (size_t)slab * (size_t)t->V * 4));
        cudaError_t e = cudaSuccess;
        for (int64_t r0 = 0; r0 < rows && e == cudaSuccess; r0 += slab) {
            const int32_t nr = (int32_t)(rows - r0 < slab ? rows - r0 : slab);
            const int32_t q_lo = state_lo + (int32_t)r0;
            // grid x = tiles of 32 tokens, y = tiles of 32 states (tiles start at multiples of 32;
            // a slab has at most a few hundred of them)
            const int32_t q_tile0 = q_lo / 32;
            const uint32_t s_tiles = (uint32_t)((q_lo + nr + 31) / 32 - q_tile0);
            const uint32_t v_tiles = (uint32_t)((t->V + 31) / 32);
            dim3 grid(v_tiles, s_tiles), block(32, 8);
            if (t->wide)
                table_decode_kernel<uint32_t><<<grid, block, 0, (cudaStream_t)cuda_stream>>>(
                    (const uint32_t *)t->next, t->lds, t->V, q_lo, nr, q_tile0, t->n_states,
                    t->code_shift, t->renumbered ? t->rank : nullptr,
                    t->renumbered ? t->unrank : nullptr, stage, CSTR_OOB_RECORD());
            else
                table_decode_kernel<uint16_t><<<grid, block, 0, (cudaStream_t)cuda_stream>>>(
                    (const uint16_t *)t->next, t->lds, t->V, q_lo, nr, q_tile0, t->n_states,
                    t->code_shift, t->renumbered ? t->rank : nullptr,
                    t->renumbered ? t->unrank : nullptr, stage, CSTR_OOB_RECORD());
            e = cudaGetLastError();
            if (e == cudaSuccess)
                e = cudaMemcpyAsync(next_host + r0 * t->V, stage, (size_t)nr * (size_t)t->V * 4,
                                    cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream);
            if (e == cudaSuccess)
                e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
        }
        cudaFree(stage);
        if (e != cudaSuccess)
            return cstr_fail(CSTR_ERR_CUDA, "cstr_table_download: %s", cudaGetErrorString(e));
    }
    return CSTR_OK;
}

// ------------------------------------------------------------ workspace

extern "C" void cstr_free_workspace(cstr_workspace_t *ws)
{
    if (!ws)
        return;
    cudaFree(ws->cell);
    cudaFree(ws->ticket);
    cudaFree(ws->counters);
    if (ws->host_ready) {
        cudaStreamDestroy(ws->copy_stream);
        cudaStreamDestroy(ws->down_stream);
        for (int i = 0; i < CSTR_HOST_SLICES; ++i) {
            cudaEventDestroy(ws->slice_ready[i]);
            cudaEventDestroy(ws->slice_done[i]);
        }
        cudaEventDestroy(ws->inputs_free);
    }
    delete ws;
}

extern "C" int cstr_workspace_create(int32_t max_batch, cstr_workspace_t **out)
{
    if (!out)
        return cstr_fail(CSTR_ERR_NULL, "cstr_workspace_create: null pointer");
    *out = nullptr;
    if (max_batch < 1)
        return cstr_fail(CSTR_ERR_ARG, "cstr_workspace_create: max_batch = %d, need >= 1",
                         max_batch);
    cstr_workspace *ws = new (std::nothrow) cstr_workspace();
    if (!ws)
        return cstr_fail(CSTR_ERR_NOMEM, "cstr_workspace_create: out of host memory");
    memset(ws, 0, sizeof *ws);
    ws->max_batch = max_batch;
    cudaError_t e = cudaGetDevice(&ws->device);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->cell, (size_t)max_batch * 8);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->ticket, (size_t)max_batch * 4);
    if (e == cudaSuccess)
        e = cudaMalloc((void **)&ws->counters, 16);
    if (e == cudaSuccess)
        e = cudaMemset(ws->cell, 0, (size_t)max_batch * 8);
    if (e == cudaSuccess)
        e = cudaMemset(ws->ticket, 0, (size_t)max_batch * 4);
    if (e == cudaSuccess)
        e = cudaMemset(ws->counters, 0, 16);
    if (e != cudaSuccess) {
        int rc = cstr_fail(e == cudaErrorMemoryAllocation ? CSTR_ERR_NOMEM : CSTR_ERR_CUDA,
                           "cstr_workspace_create: %s", cudaGetErrorString(e));
        cstr_free_workspace(ws);
        return rc;
    }
    *out = ws;
    return CSTR_OK;
}

// ----------------------------------------------------------------- step

static int step_common(const cstr_table_t *const *tables, int32_t n_tables,
                       const int32_t *row_table, const void *logits, int32_t dtype, int64_t ld,
                       const float *noise, const int32_t *states, int32_t *states_out,
                       int32_t *tokens_out, void *masked_out, uint8_t *accept_out, int32_t batch,
                       cstr_workspace_t *ws, void *cuda_stream)
{
    if (batch == 0 && tables && ws && (dtype == CSTR_F32 || dtype == CSTR_BF16))
        return CSTR_OK;              // nothing to do: the per-row arrays may be empty (null)
    if (!tables || !logits || !states || !states_out || !tokens_out || !masked_out || !ws)
        return cstr_fail(CSTR_ERR_NULL, "cstr_step: null pointer");
    if (n_tables < 1 || n_tables > CSTR_MAX_TABLES)
        return cstr_fail(CSTR_ERR_ARG, "cstr_step: n_tables = %d, need 1..%d", n_tables,
                         CSTR_MAX_TABLES);
    if (dtype != CSTR_F32 && dtype != CSTR_BF16)
        return cstr_fail(CSTR_ERR_DTYPE, "cstr_step: unknown dtype %d", dtype);
    if (batch < 0)
        return cstr_fail(CSTR_ERR_ARG, "cstr_step: batch = %d", batch);
    if (batch > ws->max_batch)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_step: batch %d exceeds workspace capacity %d",
                         batch, ws->max_batch);
    int rc = cstr_check_device(ws->device, "workspace");
    if (rc)
        return rc;
    cstr_step_args a;
    memset(&a, 0, sizeof a);
    for (int32_t i = 0; i < n_tables; ++i) {
        const cstr_table *t = tables[i];
        if (!t)
            return cstr_fail(CSTR_ERR_NULL, "cstr_step: tables[%d] is null", i);
        if (t->device != ws->device)
            return cstr_fail(CSTR_ERR_DEVICE, "cstr_step: tables[%d] is on another device", i);
        if (t->n_states < 1)
            return cstr_fail(CSTR_ERR_ARG, "cstr_step: tables[%d] has not been built", i);
        if (t->V != tables[0]->V)
            return cstr_fail(CSTR_ERR_SHAPE, "cstr_step: tables[%d] has V = %d, tables[0] has %d",
                             i, t->V, tables[0]->V);
        a.tables[i] = t;
    }
    if (ld < tables[0]->V)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_step: ld = %lld is below V = %d", (long long)ld,
                         tables[0]->V);
    if (batch == 0)
        return CSTR_OK;
    a.n_tables = n_tables;
    a.row_table = row_table;
    a.logits = logits;
    a.dtype = dtype;
    a.ld = ld;
    a.noise = noise;
    a.states = states;
    a.states_out = states_out;
    a.tokens_out = tokens_out;
    a.masked_out = masked_out;
    a.accept_out = accept_out;
    a.batch = batch;
    a.cell = ws->cell;
    a.ticket = ws->ticket;
    a.counters = ws->counters;
    a.device = ws->device;
    return cstr_launch_step(a, (cudaStream_t)cuda_stream);
}

extern "C" int cstr_step(const cstr_table_t *const *tables, int32_t n_tables,
                         const int32_t *row_table, const void *logits, int32_t dtype, int64_t ld,
                         const float *noise, int32_t *states, int32_t *tokens_out,
                         void *masked_out, uint8_t *accept_out, int32_t batch,
                         cstr_workspace_t *ws, void *cuda_stream)
{
    return step_common(tables, n_tables, row_table, logits, dtype, ld, noise, states, states,
                       tokens_out, masked_out, accept_out, batch, ws, cuda_stream);
}

extern "C" int cstr_step_history(const cstr_table_t *const *tables, int32_t n_tables,
                                 const int32_t *row_table, const void *logits, int32_t dtype,
                                 int64_t ld, const float *noise, const int32_t *states_in,
                                 int32_t *states_out, int32_t *tokens_out, void *masked_out,
                                 uint8_t *accept_out, int32_t batch, cstr_workspace_t *ws,
                                 void *cuda_stream)
{
    return step_common(tables, n_tables, row_table, logits, dtype, ld, noise, states_in,
                       states_out, tokens_out, masked_out, accept_out, batch, ws, cuda_stream);
}

// Wait for everything cstr_step_host has in flight (uploads, kernels, downloads).
static cudaError_t host_drain(cstr_workspace *ws, cudaStream_t stream)
{
    cudaError_t e = cudaStreamSynchronize(ws->copy_stream);
    const cudaError_t e1 = cudaStreamSynchronize(stream);
    const cudaError_t e2 = cudaStreamSynchronize(ws->down_stream);
    if (e == cudaSuccess)
        e = e1;
    if (e == cudaSuccess)
        e = e2;
    return e;
}

// The step with its logits in host memory: rows are cut into slices whose
// uploads run on a copy stream ahead of the step kernels of earlier slices.
extern "C" int cstr_step_host(const cstr_table_t *const *tables, int32_t n_tables,
                              const int32_t *row_table, const void *logits_host, int32_t dtype,
                              int64_t ld, const float *noise_host, int32_t *states,
                              int32_t *tokens_host, int32_t *states_host, void *logits_dev,
                              float *noise_dev, void *masked_out, void *masked_host,
                              int32_t *tokens_dev, uint8_t *accept_out, int32_t batch,
                              cstr_workspace_t *ws, void *cuda_stream)
{
    if (!tables || !ws)
        return cstr_fail(CSTR_ERR_NULL, "cstr_step_host: null pointer");
    if (dtype != CSTR_F32 && dtype != CSTR_BF16)
        return cstr_fail(CSTR_ERR_DTYPE, "cstr_step_host: unknown dtype %d", dtype);
    if (batch < 0 || ld < 0)
        return cstr_fail(CSTR_ERR_ARG, "cstr_step_host: batch = %d, ld = %lld", batch, (long long)ld);
    if (batch == 0)
        return CSTR_OK;
    if (!logits_host || !states || !tokens_host || !logits_dev || !masked_out || !tokens_dev ||
        ((noise_host != nullptr) != (noise_dev != nullptr)))
        return cstr_fail(CSTR_ERR_NULL, "cstr_step_host: null pointer (noise needs both its host "
                         "array and its device staging array)");
    if (batch > ws->max_batch)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_step_host: batch %d exceeds workspace capacity %d",
                         batch, ws->max_batch);
    int rc = cstr_check_device(ws->device, "workspace");
    if (rc)
        return rc;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    if (!ws->host_ready) {                       // first use: streams and events, no device memory
        CSTR_CUDA_TRY(cudaStreamCreateWithFlags(&ws->copy_stream, cudaStreamNonBlocking));
        CSTR_CUDA_TRY(cudaStreamCreateWithFlags(&ws->down_stream, cudaStreamNonBlocking));
        for (int i = 0; i < CSTR_HOST_SLICES; ++i) {
            CSTR_CUDA_TRY(cudaEventCreateWithFlags(&ws->slice_ready[i], cudaEventDisableTiming));
            CSTR_CUDA_TRY(cudaEventCreateWithFlags(&ws->slice_done[i], cudaEventDisableTiming));
        }
        CSTR_CUDA_TRY(cudaEventCreateWithFlags(&ws->inputs_free, cudaEventDisableTiming));
        ws->host_ready = 1;
    }
    // uploads may start once everything enqueued so far on the caller's stream is done
    CSTR_CUDA_TRY(cudaEventRecord(ws->inputs_free, stream));
    CSTR_CUDA_TRY(cudaStreamWaitEvent(ws->copy_stream, ws->inputs_free, 0));

    const size_t esz = dtype == CSTR_BF16 ? 2 : 4;
    const int n_slices = batch < CSTR_HOST_SLICES ? batch : CSTR_HOST_SLICES;
    const int per = (batch + n_slices - 1) / n_slices;
    for (int i = 0, r0 = 0; r0 < batch; ++i, r0 += per) {
        const int rows = batch - r0 < per ? batch - r0 : per;
        const size_t off = (size_t)r0 * (size_t)ld;
        cudaError_t ce = cudaMemcpyAsync((char *)logits_dev + off * esz,
                                         (const char *)logits_host + off * esz,
                                         (size_t)rows * (size_t)ld * esz, cudaMemcpyHostToDevice,
                                         ws->copy_stream);
        if (ce == cudaSuccess && noise_host)
            ce = cudaMemcpyAsync(noise_dev + off, noise_host + off, (size_t)rows * (size_t)ld * 4,
                                 cudaMemcpyHostToDevice, ws->copy_stream);
        if (ce == cudaSuccess)
            ce = cudaEventRecord(ws->slice_ready[i], ws->copy_stream);
        if (ce == cudaSuccess)
            ce = cudaStreamWaitEvent(stream, ws->slice_ready[i], 0);
        if (ce != cudaSuccess) {
            host_drain(ws, stream);
            return cstr_fail(CSTR_ERR_CUDA, "cstr_step_host: %s", cudaGetErrorString(ce));
        }
        cstr_workspace sub = *ws;                // this slice's rows of the scratch
        sub.cell += r0;
        sub.ticket += r0;
        sub.max_batch = rows;
        rc = step_common(tables, n_tables, row_table ? row_table + r0 : nullptr,
                         (const char *)logits_dev + off * esz, dtype, ld,
                         noise_dev ? noise_dev + off : nullptr, states + r0, states + r0,
                         tokens_dev + r0, (char *)masked_out + off * esz,
                         accept_out ? accept_out + r0 : nullptr, rows, &sub, stream);
        if (rc == CSTR_OK && masked_host) {      // this slice's penalised logits go down on a third
            cudaError_t e = cudaEventRecord(ws->slice_done[i], stream);     // stream, beside the uploads
            if (e == cudaSuccess)
                e = cudaStreamWaitEvent(ws->down_stream, ws->slice_done[i], 0);
            if (e == cudaSuccess)
                e = cudaMemcpyAsync((char *)masked_host + off * esz, (const char *)masked_out + off * esz,
                                    (size_t)rows * (size_t)ld * esz, cudaMemcpyDeviceToHost,
                                    ws->down_stream);
            if (e != cudaSuccess)
                rc = cstr_fail(CSTR_ERR_CUDA, "cstr_step_host: %s", cudaGetErrorString(e));
        }
        if (rc) {
            host_drain(ws, stream);
            return rc;
        }
    }
    cudaError_t e = cudaMemcpyAsync(tokens_host, tokens_dev, (size_t)batch * 4,
                                    cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess && states_host)
        e = cudaMemcpyAsync(states_host, states, (size_t)batch * 4, cudaMemcpyDeviceToHost, stream);
    // every exit, failures included, waits for all three streams: the caller's host
    // buffers must not be in use by a copy once the call has returned
    const cudaError_t e2 = host_drain(ws, stream);
    if (e == cudaSuccess)
        e = e2;
    if (e != cudaSuccess)
        return cstr_fail(CSTR_ERR_CUDA, "cstr_step_host: %s", cudaGetErrorString(e));
    return CSTR_OK;
}

extern "C" int cstr_accept_draft(const int32_t *draft_tokens, const int32_t *target_tokens,
                                 const int32_t *target_states, int32_t k, int32_t batch,
                                 int32_t *n_accepted, int32_t *out_tokens, int32_t *states,
                                 void *cuda_stream)
{
    if (!target_tokens || !target_states || !n_accepted || !out_tokens || !states ||
        (k > 0 && !draft_tokens))
        return cstr_fail(CSTR_ERR_NULL, "cstr_accept_draft: null pointer");
    if (k < 0 || batch < 0)
        return cstr_fail(CSTR_ERR_ARG, "cstr_accept_draft: k = %d, batch = %d", k, batch);
    if (batch == 0)
        return CSTR_OK;
    return cstr_launch_accept(draft_tokens, target_tokens, target_states, k, batch, n_accepted,
                              out_tokens, states, (cudaStream_t)cuda_stream);
}

extern "C" int cstr_step_status(cstr_workspace_t *ws, void *cuda_stream, int64_t *bad_state_rows,
                                int64_t *empty_mask_rows)
{
    if (!ws)
        return cstr_fail(CSTR_ERR_NULL, "cstr_step_status: null workspace");
    int rc = cstr_check_device(ws->device, "workspace");
    if (rc)
        return rc;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    unsigned long long host[2] = {0, 0};
    CSTR_CUDA_TRY(cudaMemcpyAsync(host, ws->counters, 16, cudaMemcpyDeviceToHost, stream));
    CSTR_CUDA_TRY(cudaMemsetAsync(ws->counters, 0, 16, stream));
    CSTR_CUDA_TRY(cudaStreamSynchronize(stream));
    if (bad_state_rows)
        *bad_state_rows = (int64_t)host[0];
    if (empty_mask_rows)
        *empty_mask_rows = (int64_t)host[1];
    return CSTR_OK;
}
