// Token-table builder: next[v][q] = delta*(q, bytes(v)) and the allowed-token
// bitmask, for every DFA state q and vocabulary token v (Algorithm 1 composed
// with the DFA as in Algorithm 2; Theorem 2 fixes the meaning).
//
// The detokenizing transducer of Algorithm 1 has a compact, trie-like form in
// which tokens share the chain of their common prefix (Section 2.3, Figure 4).
// The builder walks exactly that trie: tokens come in lexicographic order with
// the length of the prefix each shares with its predecessor, and a warp that
// owns a block of DFA states (one or more states per lane) keeps, per depth of
// the current trie path, the state every lane has reached.  A token then costs
// only the lookups of the bytes it does not share with the previous token.
//
//   - lane = state: every lane of a warp reads the same token, so there is no
//     divergence on token length, and all control flow is warp-uniform;
//   - the DFA is class-compressed and class-major (tt[class][slot]) with a
//     self-looping dead sink, and its entries are the byte offsets of the target
//     slots: a lookup is one add and one load, and dead walks need no branch;
//     it lives in shared memory when it fits, else it is gathered through L1/L2;
//   - a lane holds NS consecutive states (NS = 1, 2, 4 or 8) and stores their
//     next-state entries with one vector store into the token's row;
//     validity goes out as NS ballot words per (token, warp), which a second
//     kernel bit-transposes into the state-major mask the step streams.
#include "cstr_internal.cuh"

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kDepth = CSTR_STACK_DEPTH;
constexpr int kDedupMaxClasses = 16;    // duplicate-column pass: automata with at most this many
constexpr int kDedupMinTokens = 8192;   // byte classes, vocabularies of at least this many tokens
constexpr int kDedupMinStates = 2048;   // and enough states for the walk to outweigh the extra passes

#ifdef CSTR_TESTING
// Checking build only: the duplicate-column pass keeps this many bits of its
// hash, so that tests can force collisions and exercise the exact comparison
// that makes grouping safe.  The release library has no such switch.
unsigned long long g_test_hash_keep = ~0ull;
#endif

struct BuildParams {
    const void *tt;            // [n_classes][row]
    const uint8_t *cls;        // [256]
    const uint8_t *accept;     // [n_states], by the caller's state ids
    const int32_t *unrank;     // internal id -> caller's id, or null (identity)
    const uint4 *desc;         // [V] sorted tokens
    const uint32_t *pre4;      // [V] first 4 bytes of each sorted token (little endian), or null
    const uint8_t *bytes;      // raw vocabulary bytes
    const uint32_t *off;       // [V + 1]
    void *next;                // [V][lds]
    uint32_t *maskT;           // [V][ldb]
    unsigned lds, ldb;         // row pitches of next (entries) and maskT (words)
    int row;                   // entries per class row of tt
    int n_states, n_classes, V, eos_id;
    int tokens_per_cta;
    int warps_s;               // warps of a CTA that split its states ...
    int warps_t;               // ... times warps that split its token chunk
    int slice_tokens;          // pruning walks: tokens per unit of work drawn by a warp
    // extents, for the checking build's range checks (see CSTR_INB)
    unsigned long long *oob;   // bounds record, null in the release build
    long long tt_bytes;        // bytes of the class-major DFA table
    long long bytes_len;       // readable vocabulary bytes
    long long mask_words;      // words of the state-major mask
    // duplicate-column pass: desc lists one representative per class string and
    // its length is only known on the device
    const int32_t *count_dev;  // null: desc holds all V tokens
    const uint32_t *reptok;    // [V] representative token id per token id, or null
};

// NS consecutive table entries per lane travel as one aligned unit (one vector
// load / store).  Entries are handled as unsigned values (uint16 / uint32),
// which keeps packing and unpacking plain bit operations.
template <int BYTES>
struct Unit;
template <> struct Unit<2> { typedef unsigned short type; };
template <> struct Unit<4> { typedef unsigned int type; };
template <> struct Unit<8> { typedef uint2 type; };
template <> struct Unit<16> { typedef uint4 type; };

template <int ESZ, int NS>
__device__ __forceinline__ typename Unit<ESZ * NS>::type pack_entries(const unsigned (&v)[NS])
{
    typename Unit<ESZ * NS>::type u;
    if constexpr (ESZ == 2) {
        if constexpr (NS == 1) u = (unsigned short)v[0];
        if constexpr (NS == 2) u = v[0] | (v[1] << 16);            // values are below 2^16
        if constexpr (NS == 4) u = make_uint2(v[0] | (v[1] << 16), v[2] | (v[3] << 16));
        if constexpr (NS == 8) u = make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16),
                                              v[4] | (v[5] << 16), v[6] | (v[7] << 16));
    } else {
        if constexpr (NS == 1) u = v[0];
        if constexpr (NS == 2) u = make_uint2(v[0], v[1]);
        if constexpr (NS == 4) u = make_uint4(v[0], v[1], v[2], v[3]);
    }
    return u;
}

template <int ESZ, int NS>
__device__ __forceinline__ void unpack_entries(typename Unit<ESZ * NS>::type u, unsigned (&v)[NS])
{
    if constexpr (ESZ == 2) {
        if constexpr (NS == 1) v[0] = u;
        if constexpr (NS == 2) { v[0] = u & 0xffffu; v[1] = u >> 16; }
        if constexpr (NS == 4) { v[0] = u.x & 0xffffu; v[1] = u.x >> 16; v[2] = u.y & 0xffffu; v[3] = u.y >> 16; }
        if constexpr (NS == 8) {
            v[0] = u.x & 0xffffu; v[1] = u.x >> 16; v[2] = u.y & 0xffffu; v[3] = u.y >> 16;
            v[4] = u.z & 0xffffu; v[5] = u.z >> 16; v[6] = u.w & 0xffffu; v[7] = u.w >> 16;
        }
    } else {
        if constexpr (NS == 1) v[0] = u;
        if constexpr (NS == 2) { v[0] = u.x; v[1] = u.y; }
        if constexpr (NS == 4) { v[0] = u.x; v[1] = u.y; v[2] = u.z; v[3] = u.w; }
    }
}

// ST: entry type of the DFA table; NT: entry type of next; NS: states per lane;
// SMEM: the class-major DFA table is staged in shared memory; PRUNE: skip the
// walks below a trie node at which all of the warp's states are dead.
// Lane l of the warp that owns states [q0, q0 + 32 NS) holds the NS consecutive
// states q0 + NS l + j.  Ballot j therefore carries state q0 + NS l + j in bit l;
// it is stored as word (q0 / 32 + j) of the token's maskT row and un-permuted
// by the transpose kernel.
template <typename ST, typename NT, int NS, bool SMEM, bool PRUNE>
__global__ void __launch_bounds__(NS == 8 ? 1024 : 512)
build_trie_kernel(const __grid_constant__ BuildParams p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    constexpr int ESZ = (int)sizeof(ST);
    typedef typename Unit<ESZ>::type SU;                        // unsigned view of a table entry
    typedef typename Unit<ESZ * NS>::type SPack;
    typedef typename Unit<sizeof(NT) * NS>::type NPack;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // Every state id below is a "code": the byte offset of the state's slot in
    // a class row, ESZ * PERM(state).  Table entries hold codes, so a lookup is
    // one add and one load; next[] stores codes too (decoded where it is read).
    const unsigned sink = (unsigned)CSTR_PERM(p.n_states) * ESZ;

    // shared memory: [row byte offset per byte value: 256 x u32]
    //                [stack: nwarps x (kDepth+1) x 32 SPack][table]
    uint32_t *s_rowoff = (uint32_t *)smem;
    SPack *s_stack = (SPack *)(smem + 1024) + (size_t)warp * (kDepth + 1) * 32 + lane;
    const unsigned char *s_tt = smem + 1024 + (size_t)nwarps * (kDepth + 1) * 32 * sizeof(SPack);
    __shared__ int s_unit_counter;
    int *const s_unit = &s_unit_counter;
    if (threadIdx.x == 0)
        *s_unit = 0;
    for (int i = threadIdx.x; i < 256; i += blockDim.x)
        s_rowoff[i] = (uint32_t)p.cls[i] * (uint32_t)p.row * ESZ;
    if (SMEM) {
        const int n16 = (int)((long long)p.n_classes * p.row * ESZ / 16);
        const uint4 *src = (const uint4 *)p.tt;
        uint4 *dst = (uint4 *)s_tt;      // row is a multiple of 256 entries: whole 16-byte units
        for (int i = threadIdx.x; i < n16; i += blockDim.x)
            dst[i] = __ldg(src + i);
    }
    __syncthreads();
    const unsigned char *g_tt = (const unsigned char *)p.tt;

    int n_tokens = p.V, tokens_per_cta = p.tokens_per_cta;
    if (p.count_dev) {                                   // representatives only: equal shares
        n_tokens = *p.count_dev;
        tokens_per_cta = (n_tokens + (int)gridDim.y - 1) / (int)gridDim.y;
    }
    const int c_begin = blockIdx.y * tokens_per_cta;
    const int c_end = min(n_tokens, c_begin + tokens_per_cta);

    // One unit of work: the warp takes the 32 NS states of state block warp_s of
    // this CTA through the sorted tokens [t_begin, t_end).
    auto walk = [&](const int warp_s, const int t_begin, const int t_end) {
    const int q0 = (blockIdx.x * p.warps_s + warp_s) * NS * 32;
    if (q0 >= p.n_states || t_begin >= t_end)
        return;                                          // whole warp out of range
    const int qbase = q0 + NS * lane;
    unsigned cur[NS], sinks[NS];
    unsigned accbits = 0;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        const bool in = qbase + j < p.n_states;       // the kernel's states are internal ids
        if (p.eos_id >= 0)                            // accept flags only matter for an EOS token
            accbits |= (unsigned)(in && p.accept[p.unrank ? p.unrank[qbase + j] : qbase + j] != 0) << j;
        cur[j] = in ? (unsigned)CSTR_PERM(qbase + j) * ESZ : sink;
        sinks[j] = sink;
    }
    const NPack dead_out = pack_entries<sizeof(NT), NS>(sinks);
    __syncwarp();                                        // the previous unit's stack reads are done
    s_stack[0] = pack_entries<ESZ, NS>(cur);             // depth 0: the states themselves
    __syncwarp();
    NT *const next_lane = (NT *)p.next + qbase;
    uint32_t *const maskT_warp = p.maskT + (q0 >> 5);
    const unsigned char *const tbase = SMEM ? s_tt : g_tt;

    // One byte of the walk for the lane's NS states: dst = delta(src, b).
    auto step = [&](const unsigned (&src)[NS], unsigned (&dst)[NS], unsigned b) {
        const unsigned char *rowp = tbase + s_rowoff[b];
#pragma unroll
        for (int j = 0; j < NS; ++j) {
            if (!CSTR_INB(p.oob, (long long)s_rowoff[b] + src[j], p.tt_bytes, CSTR_SITE_BUILD_TT))
                dst[j] = sink;
            else if (SMEM)
                dst[j] = (unsigned)*(const SU *)(rowp + src[j]);
            else
                dst[j] = (unsigned)__ldg((const SU *)(rowp + src[j]));
        }
    };
    // Every state of the warp sits in the sink (lanes past the last state always do).
    auto all_dead = [&](const unsigned (&st)[NS]) -> bool {
        unsigned x = 0u;
#pragma unroll
        for (int j = 0; j < NS; ++j)
            x |= st[j] ^ sink;
        return __all_sync(kFull, x == 0u);
    };

    // A token's outputs: the lane's entries of the token's row of next, and one
    // ballot word per state slot of the lane.  "No edge" goes out as the sink's
    // own code (decoded to -1 by readers), so live walks are stored as they
    // are; lanes past the last state sit in the sink from the start.
    NPack outp = dead_out;
    uint32_t words[NS];
    auto outputs_of = [&](const unsigned (&st)[NS]) {
        outp = pack_entries<sizeof(NT), NS>(st);
#pragma unroll
        for (int j = 0; j < NS; ++j)
            words[j] = __ballot_sync(kFull, st[j] != sink);
    };
    auto store_outputs = [&](unsigned tok) {
        if (!CSTR_INB(p.oob, tok, p.V, CSTR_SITE_BUILD_NEXT) ||
            !CSTR_INB(p.oob, qbase + NS - 1, p.lds, CSTR_SITE_BUILD_NEXT) ||
            !CSTR_INB(p.oob, (q0 >> 5) + NS - 1, p.ldb, CSTR_SITE_BUILD_MASKT))
            return;
        // lds is a multiple of 256 states: the whole unit is inside the token's row
        *(NPack *)(next_lane + (unsigned long long)tok * p.lds) = outp;
        if (lane == 0) {                 // ballots are warp-uniform; (q0 >> 5) + NS <= lds / 32 < ldb
            uint32_t *mrow = maskT_warp + (unsigned long long)tok * p.ldb;          // NS-word aligned
            if constexpr (NS == 1) *mrow = words[0];
            if constexpr (NS == 2) *(uint2 *)mrow = make_uint2(words[0], words[1]);
            if constexpr (NS >= 4) *(uint4 *)mrow = make_uint4(words[0], words[1], words[2], words[3]);
            if constexpr (NS == 8) *(uint4 *)(mrow + 4) = make_uint4(words[4], words[5], words[6], words[7]);
        }
    };

    // par[] = the lane's states after the first pd bytes of the current trie
    // path, kept in registers: consecutive tokens are mostly siblings (same
    // shared prefix, one byte of their own), which then cost one lookup round
    // and no stack traffic.  The shared-memory stack holds the states at depth
    // j only while a later token can still resume there, i.e. for j up to the
    // NEXT token's shared prefix (known from the prefetched descriptor): leaves,
    // the bulk of the tokens, store nothing.
    // PRUNE (sparse automata): once every state of the warp is dead at some
    // depth of the path, every token below that trie node is dead in the whole
    // warp; such tokens get their dead outputs without any lookup until a token
    // resumes above that depth (the sparse composition touches live edges only).
    unsigned par[NS];
#pragma unroll
    for (int j = 0; j < NS; ++j)
        par[j] = cur[j];
    int pd = 0;
    int dead_from = 0x7fffffff;                          // depth at which the path died
    bool first = true;      // the chunk's first token is walked from the root, all its bytes
                            // from the vocabulary (its descriptor starts at a prefix shared
                            // with a token of another chunk)
    // The next token's descriptor is loaded one token ahead (same address in every
    // lane).  Past the end of the walk: y = all ones.  (Handing descriptors around
    // by shuffles from one coalesced load per 32 tokens was measured: more
    // instructions, no gain.)
    const uint4 no_desc = make_uint4(0u, 0xffffffffu, 0u, 0u);
    auto fetch = [&](int idx) -> uint4 {
        return (idx < t_end && CSTR_INB(p.oob, idx, n_tokens, CSTR_SITE_BUILD_VOCAB))
                   ? __ldg(p.desc + idx) : no_desc;
    };
    // Descriptors are loaded two tokens ahead: the NEXT token's shared prefix is
    // needed while the current token is walked, so one token ahead would put the
    // load latency back on the critical path.
    uint4 d = fetch(t_begin), dn = fetch(t_begin + 1);
    // The walk's first token starts at the root, but its descriptor carries its bytes
    // only from its shared prefix on; the (at most kDepth) bytes before that come from
    // pre4, loaded here beside the descriptors, so that no dependent load sits in the
    // first token's walk.
    const uint32_t first_pre = (PRUNE && p.pre4) ? __ldg(p.pre4 + t_begin) : 0u;
    const int first_tsh = (PRUNE && p.pre4) ? (int)(d.y >> 24) : 0;
#pragma unroll 1
    for (int i = t_begin; i < t_end; ++i) {
        uint4 dnn = fetch(i + 2);
        const int nsh = dn.y == 0xffffffffu ? 0 : (int)(dn.y >> 24);    // at most kDepth
        const unsigned tok = d.x;
        const int n = (int)(d.y & 0xffffffu);
        const int sh = first ? 0 : (int)(d.y >> 24);
        const bool is_eos = (int)tok == p.eos_id;
        bool dead = PRUNE && sh >= dead_from;
        if (!dead) {
            if (PRUNE)
                dead_from = 0x7fffffff;
            if (sh != pd && CSTR_INB(p.oob, sh, kDepth + 1, CSTR_SITE_BUILD_STACK)) {   // resume at the shared prefix
                unpack_entries<ESZ, NS>(s_stack[sh * 32], par);
                pd = sh;
            }
            const int m = n - sh;                        // bytes of its own
            if (m == 0) {                                // same string as its predecessor (or empty)
                outputs_of(par);
            } else {
                // (bz, bw, bx) hold the token's next `inl` bytes from position sh on: d.z / d.w
                // carry 8 bytes from the shared prefix on; for a walk's first token (sh = 0)
                // the up to kDepth bytes before that come from pre4.  Whatever lies beyond
                // comes from the vocabulary.
                unsigned bz = d.z, bw = d.w, bx = 0u;
                int inl = 8;
                if (first) {
                    if (PRUNE && p.pre4) {       // (only the pruning walks, whose units are short,
                                                 // gain from it; elsewhere it only costs instructions)
                        const int tsh = first_tsh;           // 0 .. kDepth
                        const unsigned long long tail = ((unsigned long long)d.w << 32) | d.z;
                        const unsigned long long lo = tsh ? ((tail << (8 * tsh)) | first_pre) : tail;
                        bz = (unsigned)lo;
                        bw = (unsigned)(lo >> 32);
                        bx = tsh ? (unsigned)(tail >> (64 - 8 * tsh)) : 0u;
                        inl = 8 + tsh;
                    } else {
                        inl = 0;
                    }
                }
                uint32_t gb = 0u;
                if (m > inl && CSTR_INB(p.oob, tok, p.V, CSTR_SITE_BUILD_VOCAB))
                    gb = __ldg(p.off + tok) + (uint32_t)sh;
                // (a token's bytes end inside the vocabulary: gb + m <= bytes_len)
                const bool bytes_ok = CSTR_INB(p.oob, (long long)gb + m - 1, p.bytes_len, CSTR_SITE_BUILD_VOCAB);
                auto byte_at = [&](int k) -> unsigned {  // own byte k of the token (position sh + k)
                    if (PRUNE) {
                        if (k < 8 && k < inl)
                            return __byte_perm(bz, bw, (unsigned)k) & 0xffu;
                        if (k < inl)
                            return __byte_perm(bx, 0u, (unsigned)(k - 8)) & 0xffu;
                    } else if (k < inl) {                // inl is 0 or 8 here
                        return __byte_perm(bz, bw, (unsigned)k) & 0xffu;
                    }
                    return bytes_ok ? (unsigned)__ldg(p.bytes + gb + k) : 0u;
                };
                step(par, cur, byte_at(0));
                if (PRUNE && all_dead(cur)) {
                    dead_from = sh + 1;
                    dead = true;
                }
                if (m > 1 && !dead) {
#pragma unroll 1
                    for (int k = 1; k < m; ++k) {
                        if (sh + k <= nsh && CSTR_INB(p.oob, sh + k, kDepth + 1, CSTR_SITE_BUILD_STACK))
                            s_stack[(sh + k) * 32] = pack_entries<ESZ, NS>(cur);
                        step(cur, cur, byte_at(k));
                        if (PRUNE && all_dead(cur)) {
                            dead_from = sh + k + 1;
                            dead = true;
                            break;
                        }
                    }
                }
                if (!dead) {
                    outputs_of(cur);
                    if (n <= nsh && CSTR_INB(p.oob, n, kDepth + 1, CSTR_SITE_BUILD_STACK)) {   // the next token extends (or repeats) this one
                        s_stack[n * 32] = pack_entries<ESZ, NS>(cur);
#pragma unroll
                        for (int j = 0; j < NS; ++j)
                            par[j] = cur[j];
                        pd = n;
                    }
                }
            }
        }
        if (dead) {
            outp = dead_out;
#pragma unroll
            for (int j = 0; j < NS; ++j)
                words[j] = 0u;
        }
        if (n == 0 || is_eos) {          // empty token: no edge.  EOS: allowed exactly in
            outp = dead_out;             // accepting states, and it finishes the row.
#pragma unroll
            for (int j = 0; j < NS; ++j)
                words[j] = __ballot_sync(kFull, is_eos && ((accbits >> j) & 1u));
        }
        store_outputs(tok);
        first = false;
        // Runs of tokens with these same outputs: tokens that repeat this one (same
        // length, all of it shared: only strings of at most kDepth bytes can say so),
        // and, below a trie node at which the whole warp is dead, every token of the
        // subtree.  The run's descriptors come 32 at a time, one per lane (a single
        // load latency per block instead of one per token); a ballot finds where the
        // run ends and the token ids are handed round by shuffles.
        if (!is_eos) {
            const unsigned same = (unsigned)n | ((unsigned)n << 24);
            const bool by_death = PRUNE && dead;
            auto in_run = [&](const uint4 &x) -> bool {
                if (x.y == 0xffffffffu || (int)x.x == p.eos_id)
                    return false;
                return by_death ? (int)(x.y >> 24) >= dead_from : (n <= kDepth && x.y == same);
            };
            if (in_run(dn)) {
                int j = i + 1;                               // first token of the run
                for (;;) {
                    const uint4 mine = fetch(j + lane);
                    const unsigned not_in = ~__ballot_sync(kFull, in_run(mine));
                    const int len = not_in == 0u ? 32 : __ffs((int)not_in) - 1;
                    for (int t = 0; t < len; ++t)
                        store_outputs(__shfl_sync(kFull, mine.x, t));
                    j += len;
                    if (len < 32) {                          // lane `len` holds the token after the run
                        dn = make_uint4(__shfl_sync(kFull, mine.x, len), __shfl_sync(kFull, mine.y, len),
                                        __shfl_sync(kFull, mine.z, len), __shfl_sync(kFull, mine.w, len));
                        break;
                    }
                }
                i = j - 1;
                dnn = fetch(i + 2);
            }
        }
        d = dn;
        dn = dnn;
    }
    };  // walk

    if (!PRUNE) {
        // static shares: state block = warp % warps_s, token slice = warp / warps_s
        const int per_t = (c_end - c_begin + p.warps_t - 1) / p.warps_t;
        const int t_begin = c_begin + (warp / p.warps_s) * per_t;
        walk(warp % p.warps_s, t_begin, min(c_end, t_begin + per_t));
    } else {
        // Pruned walks differ widely in cost (a warp whose states all die early
        // flies through its tokens), so the warps of the CTA draw (state block,
        // token slice) units from a counter.  State blocks come in ascending
        // order: the states that allow many bytes are numbered first, so the
        // long units start first.
        // The slices of a CTA are spread over the whole sorted token list (slice
        // y, y + gridDim.y, ...): the cost of a stretch of tokens varies along the
        // list (runs of repeated one-byte tokens are nearly free, long tokens are
        // not), and a contiguous chunk per CTA would leave some SMs idle early.
        const int slice = p.slice_tokens;
        const int total_slices = (n_tokens + slice - 1) / slice;
        const int n_slices = total_slices > (int)blockIdx.y
                                 ? (total_slices - (int)blockIdx.y + (int)gridDim.y - 1) / (int)gridDim.y : 0;
        const int n_units = p.warps_s * n_slices;
        for (;;) {
            int unit = 0;
            if (lane == 0)
                unit = atomicAdd(s_unit, 1);
            unit = __shfl_sync(kFull, unit, 0);
            if (unit >= n_units)
                break;
            const int ws = unit / n_slices;
            const int t_begin = ((int)blockIdx.y + (unit - ws * n_slices) * (int)gridDim.y) * slice;
            walk(ws, t_begin, min(n_tokens, t_begin + slice));
        }
    }
}

// The table's own copy of the automaton's accept flags and (for a renumbered
// automaton) of rank + unrank, which sit back to back in both the DFA and the
// table.  A few KB: separate device-to-device copies or a kernel of their own
// would cost several microseconds of every build, so the first CTA of the
// mask transpose does it on the side; builds without a transpose pass launch
// table_meta_kernel.
struct MetaCopy {
    const uint8_t *accept_src;
    uint8_t *accept_dst;
    int n_states;
    const int32_t *rank_src;
    int32_t *rank_dst;
    int rank_words;            // 2 (n_states + 1), or 0 for the identity numbering
};

__device__ __forceinline__ void meta_copy(const MetaCopy &m, int first, int stride)
{
    for (int i = first; i < m.n_states; i += stride)
        m.accept_dst[i] = m.accept_src[i];
    for (int i = first; i < m.rank_words; i += stride)
        m.rank_dst[i] = m.rank_src[i];
}

__global__ void __launch_bounds__(256)
table_meta_kernel(const MetaCopy m)
{
    meta_copy(m, blockIdx.x * 256 + threadIdx.x, gridDim.x * 256);
}

// mask[q][w] bit t = validity of token 32 w + t in state q, gathered from the
// per-token ballot words: 32 x 32 bit-matrix transposes.  A CTA takes 1,024
// tokens (32 mask words) x 8 ballot words.  Warp j handles ballot word sb0 + j;
// lane l takes the 32 tokens of mask word w0 + l into registers, transposes the
// 32 x 32 bit block in registers (no shuffles), and for each of the 32 states
// the warp stores 32 consecutive mask words of that state's row (128 bytes).
// Ballot word k of a block of 32 NS states holds state NS l + k of the block
// in bit l.  Ballot rows are in the builder's internal state numbering.
__global__ void __launch_bounds__(256)
mask_transpose_kernel(const uint32_t *__restrict__ maskT, long long ldb, uint32_t *__restrict__ mask,
                      long long ldw, int n_states, int V, int ns,
                      const uint32_t *__restrict__ reptok, const int32_t *__restrict__ unrank,
                      long long mask_words, unsigned long long *oob, const MetaCopy meta)
{
    // one padding word per 32 tokens: lane l then reads word 33 l + r, free of bank conflicts
    __shared__ uint32_t tile[8][1024 + 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (blockIdx.x == 0 && blockIdx.y == 0)
        meta_copy(meta, threadIdx.x, 256);
    // x = group of 32 mask words, y = group of 8 ballot words: CTAs launched
    // together write neighbouring 128-byte pieces of the same mask rows (the four
    // CTAs that read the 32-byte quarters of one maskT line meet again in L2)
    const int w0 = blockIdx.x * 32;
    const int sb0 = blockIdx.y * 8;
    // four tokens per thread; all row indices first, then all row loads, so that
    // the dependent loads of the four tokens overlap
    long long rowid[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const long long tokid = (long long)w0 * 32 + threadIdx.x + 256 * k;
        // after a duplicate-column pass only the representatives' rows were written
        rowid[k] = tokid < V ? (reptok ? (long long)__ldg(reptok + tokid) : tokid) : -1;
    }
    uint4 lo[4], hi[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        lo[k] = hi[k] = make_uint4(0u, 0u, 0u, 0u);
        if (rowid[k] >= 0 && CSTR_INB(oob, rowid[k], V, CSTR_SITE_TRANSPOSE) &&
            CSTR_INB(oob, sb0 + 7, ldb, CSTR_SITE_TRANSPOSE)) {
            const uint4 *src = (const uint4 *)(maskT + rowid[k] * ldb + sb0);   // ldb, sb0 multiples of 8
            lo[k] = __ldg(src);
            hi[k] = __ldg(src + 1);
        }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int t = threadIdx.x + 256 * k;
        const int at = t + (t >> 5);
        tile[0][at] = lo[k].x; tile[1][at] = lo[k].y; tile[2][at] = lo[k].z; tile[3][at] = lo[k].w;
        tile[4][at] = hi[k].x; tile[5][at] = hi[k].y; tile[6][at] = hi[k].z; tile[7][at] = hi[k].w;
    }
    __syncthreads();
    const int sbw = sb0 + warp;
    const int first_state = (sbw / ns) * (ns * 32) + (sbw % ns);
    if (first_state >= n_states)
        return;
    uint32_t x[32];                                      // x[r]: token 32 (w0 + lane) + r, bit = state slot
#pragma unroll
    for (int r = 0; r < 32; ++r)
        x[r] = tile[warp][33 * lane + r];
    // 32 x 32 bit transpose by block swaps of 16, 8, 4, 2 and 1 bits; the two
    // coarse stages move whole bytes, which is one byte permute per word
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const uint32_t a = x[k], b = x[k + 16];
        x[k] = __byte_perm(a, b, 0x5410);            // low half of a, low half of b
        x[k + 16] = __byte_perm(a, b, 0x7632);       // high half of a, high half of b
    }
#pragma unroll
    for (int k = 0; k < 32; ++k) {
        if ((k & 8) == 0) {
            const uint32_t a = x[k], b = x[k + 8];
            x[k] = __byte_perm(a, b, 0x6240);        // bytes a0 b0 a2 b2
            x[k + 8] = __byte_perm(a, b, 0x7351);    // bytes a1 b1 a3 b3
        }
    }
    uint32_t m = 0x0f0f0f0fu;
#pragma unroll
    for (int j = 4; j >= 1; j >>= 1) {
#pragma unroll
        for (int k = 0; k < 32; ++k) {
            if ((k & j) == 0) {
                const uint32_t t = ((x[k] >> j) ^ x[k + j]) & m;
                x[k] ^= t << j;
                x[k + j] ^= t;
            }
        }
        m ^= m << (j >> 1);
    }
    // now x[s]: state slot s, bit = token: mask word w0 + lane of (internal) state
    // first_state + ns s; the mask rows are indexed by the caller's state ids
    uint32_t *dst = mask + w0 + lane;                                        // ldw multiple of 32
#pragma unroll
    for (int sl = 0; sl < 32; ++sl) {
        const int qi = first_state + ns * sl;
        if (qi < n_states) {                             // warp-uniform
            const long long row = unrank ? unrank[qi] : qi;
            if (CSTR_INB(oob, row * ldw + w0 + lane, mask_words, CSTR_SITE_TRANSPOSE))
                dst[row * ldw] = x[sl];
        }
    }
}

// Terminal-label edges (wildcards matched by pre-computed token sets): for
// every state that has some, every token without an ordinary edge takes the
// terminal edge of the lowest label whose set holds it, and becomes allowed.
// One thread = one token, looping over the states with terminal edges (their
// entries of the token's row share sectors when the states are neighbours);
// the mask words are OR-ed by the warp that owns the 32 tokens, so no other
// warp touches them.
template <typename NT>
__global__ void __launch_bounds__(256)
apply_terminals_kernel(const int32_t *__restrict__ tstate, const uint32_t *__restrict__ tset,
                       const uint32_t *__restrict__ ttarget, int n_term_states, int n_labels,
                       const uint32_t *__restrict__ tsets, const uint32_t *__restrict__ off, int V,
                       int eos_id, unsigned sink, const int32_t *__restrict__ rank,
                       NT *__restrict__ next, long long lds, uint32_t *__restrict__ mask,
                       long long ldw, long long mask_words, unsigned long long *oob)
{
    const int v = blockIdx.x * 256 + threadIdx.x;
    const bool eligible = v < V && v != eos_id && off[min(v, V - 1) + 1] > off[min(v, V - 1)];
    const uint32_t mine = eligible ? tsets[v] : 0u;
    if (__ballot_sync(kFull, mine != 0u) == 0u)
        return;                                          // no token of this warp is in any set
    NT *row = next + (long long)min(v, V - 1) * lds;
    for (int i = 0; i < n_term_states; ++i) {
        const int q = tstate[i];                         // the caller's id: mask row
        const int qi = rank ? rank[q] : q;               // internal id: entry of next
        const uint32_t labels = mine & tset[i];
        bool fresh = false;
        if (labels != 0u && CSTR_INB(oob, qi, lds, CSTR_SITE_TERMINALS) && (unsigned)row[qi] == sink) {
            row[qi] = (NT)ttarget[(long long)i * n_labels + (__ffs((int)labels) - 1)];
            fresh = true;
        }
        const uint32_t word = __ballot_sync(kFull, fresh);
        if ((threadIdx.x & 31) == 0 && word != 0u &&
            CSTR_INB(oob, (long long)q * ldw + (v >> 5), mask_words, CSTR_SITE_TERMINALS))
            mask[(long long)q * ldw + (v >> 5)] |= word;
    }
}

// ---- duplicate columns -------------------------------------------------------
//
// Two tokens that read as the same string of byte classes have the same column
// of the table in every state.  For automata with few byte classes (a quoted
// string tells apart quote, backslash and "anything else") a natural vocabulary
// collapses to a few hundred class strings, so the walk runs for one
// representative per class string and the other columns are copies.
// Grouping is by a 64-bit hash in an open-addressing table, then proven by an
// exact comparison: a token whose class string differs from its group's
// representative (a hash collision) simply stays its own representative.

__device__ __forceinline__ unsigned long long class_string_hash(const uint8_t *__restrict__ cls,
                                                                const uint8_t *__restrict__ b,
                                                                unsigned n, unsigned long long keep)
{
    unsigned long long h = 0x9e3779b97f4a7c15ull ^ (unsigned long long)n;
    for (unsigned k = 0; k < n; ++k) {
        h = (h ^ (unsigned long long)cls[b[k]]) * 0x100000001b3ull;
        h ^= h >> 29;
    }
    h ^= h >> 32;
    h *= 0xd6e8feb86659fd93ull;
    h ^= h >> 32;
    return (h & keep) | 1ull;                            // 0 marks an empty slot
}

// Each group's slot ends up holding the smallest sorted index of the group.
__global__ void __launch_bounds__(256)
group_insert_kernel(const uint4 *__restrict__ desc, const uint8_t *__restrict__ bytes,
                    const uint32_t *__restrict__ off, const uint8_t *__restrict__ cls, int i_begin,
                    int i_end, int eos_id, unsigned long long *key, uint32_t *minv, uint32_t slots,
                    unsigned long long keep)
{
    const int i = i_begin + blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= i_end)
        return;
    const unsigned tok = desc[i].x;
    if ((int)tok == eos_id)
        return;                                          // the EOS column is special: never shared
    const uint32_t b0 = off[tok], b1 = off[tok + 1];
    const unsigned long long h = class_string_hash(cls, bytes + b0, b1 - b0, keep);
    uint32_t slot = (uint32_t)(h >> 20) & (slots - 1);
    for (uint32_t probe = 0; probe < slots; ++probe) {   // slots >= 4 V: an empty slot exists
        unsigned long long seen = *(volatile unsigned long long *)(key + slot);
        if (seen == 0ull)
            seen = atomicCAS(key + slot, 0ull, h);       // returns 0 if this thread claimed it
        if (seen == 0ull || seen == h) {
            // the minimum only ever falls, so a value already at or below i needs no atomic:
            // thousands of tokens share a few popular class strings
            if (*(volatile uint32_t *)(minv + slot) > (uint32_t)i)
                atomicMin(minv + slot, (uint32_t)i);
            return;
        }
        slot = (slot + 1) & (slots - 1);
    }
}

__global__ void __launch_bounds__(1024)
group_resolve_kernel(const uint4 *__restrict__ desc, const uint8_t *__restrict__ bytes,
                     const uint32_t *__restrict__ off, const uint8_t *__restrict__ cls, int V,
                     int eos_id, const unsigned long long *__restrict__ key,
                     const uint32_t *__restrict__ minv, uint32_t slots, unsigned long long keep,
                     uint32_t *__restrict__ rep, uint32_t *__restrict__ reptok,
                     int32_t *__restrict__ blk)
{
    // blocks of 1,024 sorted tokens; the block also counts its representatives (blk)
    const int i = blockIdx.x * 1024 + threadIdx.x;
    const bool in = i < V;
    const unsigned tok = in ? desc[i].x : 0u;
    uint32_t r = (uint32_t)i;
    unsigned rtok = tok;
    if (in && (int)tok != eos_id) {
        const uint32_t b0 = off[tok], n = off[tok + 1] - b0;
        const unsigned long long h = class_string_hash(cls, bytes + b0, n, keep);
        uint32_t slot = (uint32_t)(h >> 20) & (slots - 1);
        for (uint32_t probe = 0; probe < slots; ++probe) {
            const unsigned long long k = key[slot];
            if (k == h) {
                r = minv[slot];
                break;
            }
            if (k == 0ull)
                break;                                   // cannot happen after the insert pass
            slot = (slot + 1) & (slots - 1);
        }
        if (r != (uint32_t)i) {                          // prove it: same length, same classes
            rtok = desc[r].x;
            const uint32_t c0 = off[rtok], m = off[rtok + 1] - c0;
            bool same = m == n && (int)rtok != eos_id;
            for (uint32_t k = 0; same && k < n; ++k)
                same = cls[bytes[b0 + k]] == cls[bytes[c0 + k]];
            if (!same) {
                r = (uint32_t)i;
                rtok = tok;
            }
        }
    }
    if (in) {
        rep[i] = r;
        reptok[tok] = rtok;
    }
    const int n = __syncthreads_count(in && r == (uint32_t)i);
    if (threadIdx.x == 0)
        blk[blockIdx.x] = n;
}

// Representatives in sorted order: the resolve pass leaves a count per block of
// 1,024 sorted tokens; an exclusive scan of the counts, then a scatter by rank.
__global__ void __launch_bounds__(1024)
group_scan_kernel(int32_t *__restrict__ blk, int n_blocks, int32_t *__restrict__ count)
{
    __shared__ int s_sum[1024];
    const int t = threadIdx.x;
    const int per = (n_blocks + 1023) / 1024;
    const int lo = min(n_blocks, t * per), hi = min(n_blocks, lo + per);
    int sum = 0;
    for (int k = lo; k < hi; ++k)
        sum += blk[k];
    s_sum[t] = sum;
    __syncthreads();
    if (t == 0) {                                        // 1,024 partial sums: a serial scan is enough
        int acc = 0;
        for (int k = 0; k < 1024; ++k) {
            const int c = s_sum[k];
            s_sum[k] = acc;
            acc += c;
        }
        *count = acc;
    }
    __syncthreads();
    int acc = s_sum[t];
    for (int k = lo; k < hi; ++k) {
        const int c = blk[k];
        blk[k] = acc;                                    // exclusive prefix
        acc += c;
    }
}

__global__ void __launch_bounds__(1024)
group_scatter_kernel(const uint32_t *__restrict__ rep, int V, const int32_t *__restrict__ blk,
                     uint32_t *__restrict__ uniq)
{
    __shared__ int s_warp[32];
    const int i = blockIdx.x * 1024 + threadIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool flag = i < V && rep[i] == (uint32_t)i;
    const unsigned bal = __ballot_sync(kFull, flag);
    if (lane == 0)
        s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
        int v = s_warp[lane], incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(kFull, incl, o);
            if (lane >= o)
                incl += y;
        }
        s_warp[lane] = incl - v;
    }
    __syncthreads();
    if (flag)
        uniq[blk[blockIdx.x] + s_warp[warp] + __popc(bal & ((1u << lane) - 1u))] = (uint32_t)i;
}

// Trie descriptors of the representatives' own sorted list: entry k = { token id,
// length | shared prefix with representative k-1 (clipped to the walk's stack
// depth) << 24, first 8 bytes after that prefix }.
__global__ void __launch_bounds__(256)
group_desc_kernel(const uint4 *__restrict__ desc, const uint32_t *__restrict__ uniq,
                  const int32_t *__restrict__ count, const uint8_t *__restrict__ bytes,
                  const uint32_t *__restrict__ off, uint4 *__restrict__ udesc)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= *count)
        return;
    const unsigned tok = desc[uniq[k]].x;
    const uint32_t b0 = off[tok], len = off[tok + 1] - b0;
    uint32_t shared = 0;
    if (k > 0) {
        const unsigned ptok = desc[uniq[k - 1]].x;
        const uint32_t p0 = off[ptok], plen = off[ptok + 1] - p0;
        const uint32_t m = min(min(len, plen), (uint32_t)kDepth);
        while (shared < m && bytes[b0 + shared] == bytes[p0 + shared])
            ++shared;
    }
    uint32_t lo8 = 0, hi8 = 0;
    for (uint32_t j = 0; j < 8 && shared + j < len; ++j) {
        const uint32_t byte = bytes[b0 + shared + j];
        if (j < 4)
            lo8 |= byte << (8 * j);
        else
            hi8 |= byte << (8 * (j - 4));
    }
    udesc[k] = make_uint4(tok, len | (shared << 24), lo8, hi8);
}

// One CTA per token: a token that is not its own representative takes the
// representative's row of next (token-major: contiguous).
__global__ void __launch_bounds__(256)
expand_rows_kernel(const uint32_t *__restrict__ reptok, unsigned char *__restrict__ next,
                   unsigned long long next_pitch, int next_n16, int V, unsigned long long *oob)
{
    const uint32_t v = blockIdx.x;
    const uint32_t r = reptok[v];
    if (r == v || !CSTR_INB(oob, r, V, CSTR_SITE_EXPAND))
        return;
    const uint4 *src = (const uint4 *)(next + r * next_pitch);
    uint4 *dst = (uint4 *)(next + v * next_pitch);
    for (int k = threadIdx.x; k < next_n16; k += blockDim.x)
        __stcs(dst + k, __ldg(src + k));
}

// ---- small automata ----------------------------------------------------------
//
// With a handful of states the lane = state walker uses a fraction of its lanes
// and its per-token cost is all bookkeeping.  Here a lane owns a token instead and walks it from every state
// in turn, eight at a time: the byte classes of the token's first 16 bytes sit in registers,
// the class-major DFA table in shared memory, eight results at a time leave as
// one 16-byte store into the token's row of next, and the validity of a state
// over the warp's 32 tokens is one ballot = one word of mask, so no transpose
// pass is needed.  16-bit tables only.
constexpr int kLaneTokenStates = 64;   // beyond this the trie walker's shared prefixes win (measured)
constexpr int kSmallStates = 16;     // beyond this the trie walker's shared prefixes win (measured)

// Shared-memory table of the lane = token kernels.  The permuted slots of the
// global table put the states of a small automaton on a handful of banks, and
// its 512-byte rows put every class on the same ones; 32 lanes looking up
// unrelated (class, state) entries would collide there.  So a CTA stages a
// compact copy: entry [c][s], s = 0 .. n_states (the last is the sink), holds
// 2 x the plain target state, and a row takes an odd number of 32-bit words,
// which spreads the classes over the banks.  Walks run on these compact codes;
// a result is turned back into the table's permuted code when it is stored.
__host__ __device__ inline int compact_stride(int n_states)   // in 16-bit entries
{
    return 2 * (((n_states + 2) / 2) | 1);
}

__device__ __forceinline__ void stage_compact_table(const unsigned short *__restrict__ tt, int row,
                                                    int n_states, int n_classes,
                                                    unsigned short *s_tab)
{
    const int per = n_states + 1, stride = compact_stride(n_states);
    for (int i = threadIdx.x; i < n_classes * per; i += blockDim.x) {
        const int c = i / per, st = i - c * per;
        const unsigned code = __ldg(tt + (size_t)c * row + CSTR_PERM(st));
        s_tab[c * stride + st] = (unsigned short)(CSTR_UNPERM(code >> 1) << 1);
    }
}

__device__ __forceinline__ unsigned permuted_code(unsigned compact)
{
    const unsigned st = compact >> 1;
    return (unsigned)CSTR_PERM(st) << 1;
}

__global__ void __launch_bounds__(256)
build_small_kernel(const unsigned short *__restrict__ tt, const uint8_t *__restrict__ cls,
                   const uint8_t *__restrict__ accept, const uint8_t *__restrict__ bytes,
                   const uint32_t *__restrict__ off, unsigned short *__restrict__ next,
                   uint32_t *__restrict__ mask, unsigned lds, long long ldw, int row, int n_states,
                   int n_classes, int V, int W, int eos_id, long long bytes_len,
                   unsigned long long *oob)
{
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned short *s_tt = (unsigned short *)smem;            // [n_classes][compact_stride]
    uint8_t *s_cls = smem + (size_t)n_classes * compact_stride(n_states) * 2;   // [256]
    stage_compact_table(tt, row, n_states, n_classes, s_tt);
    for (int i = threadIdx.x; i < 256; i += blockDim.x)
        s_cls[i] = cls[i];
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (w >= W)
        return;
    const int v = w * 32 + lane;
    const bool in = v < V;
    const uint32_t b0 = in ? off[v] : 0u;
    int len = in ? (int)(off[v + 1] - b0) : 0;
    if (len > 0 && !CSTR_INB(oob, (long long)b0 + len - 1, bytes_len, CSTR_SITE_BUILD_VOCAB))
        len = 0;
    const bool is_eos = in && v == eos_id;
    unsigned long long c_lo = 0ull, c_hi = 0ull;              // classes of bytes 0..7 and 8..15
    for (int k = 0; k < len && k < 16; ++k) {
        const unsigned long long c = (unsigned long long)s_cls[bytes[b0 + k]] << (8 * (k & 7));
        if (k < 8)
            c_lo |= c;
        else
            c_hi |= c;
    }
    const unsigned sink = (unsigned)n_states * 2u;
    const unsigned row_bytes = (unsigned)compact_stride(n_states) * 2u;
    const unsigned char *tb = (const unsigned char *)s_tt;
    unsigned short *out = next + (unsigned long long)(in ? v : 0) * lds;
    const bool walks = in && len > 0 && !is_eos;
    for (int q0 = 0; q0 < n_states; q0 += 8) {
        // eight states side by side: one class extraction per byte, eight
        // independent shared-memory lookups (the sink maps to itself)
        unsigned cur[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            cur[j] = (walks && q0 + j < n_states) ? (unsigned)(q0 + j) * 2u : sink;
        if (walks) {
            for (int k = 0; k < len; ++k) {
                const unsigned c = k < 16 ? (unsigned)((k < 8 ? c_lo : c_hi) >> (8 * (k & 7))) & 0xffu
                                          : (unsigned)s_cls[bytes[b0 + k]];
                const unsigned char *rowp = tb + c * row_bytes;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    cur[j] = *(const unsigned short *)(rowp + cur[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int q = q0 + j;
            const bool ok = is_eos ? (q < n_states && accept[q] != 0) : cur[j] != sink;
            const unsigned word = __ballot_sync(kFull, in && ok);
            if (lane == 0 && q < n_states && CSTR_INB(oob, w, ldw, CSTR_SITE_BUILD_MASKT))
                mask[(long long)q * ldw + w] = word;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            cur[j] = permuted_code(cur[j]);
        if (in && CSTR_INB(oob, q0 + 7, lds, CSTR_SITE_BUILD_NEXT))   // lds is a multiple of 256 entries
            *(uint4 *)(out + q0) = make_uint4(cur[0] | (cur[1] << 16), cur[2] | (cur[3] << 16),
                                              cur[4] | (cur[5] << 16), cur[6] | (cur[7] << 16));
    }
}

// ---- automata of 17 to 64 states ------------------------------------------------
//
// The same lane = token walk for automata of 17 to 64 states, with two changes: a warp takes 32 tokens of EQUAL LENGTH (the vocabulary's
// by-length order), so no lane idles while a longer neighbour finishes, and a
// lane keeps its token's validity bits itself - word k of the token's maskT
// row holds states 32 k .. 32 k + 31 - for the transpose pass (one state per
// ballot word, NS = 1).  Eight states per round, one class extraction per byte,
// eight independent shared-memory lookups.
__global__ void __launch_bounds__(256)
build_lane_token_kernel(const unsigned short *__restrict__ tt, const uint8_t *__restrict__ cls,
                        const uint8_t *__restrict__ accept, const uint8_t *__restrict__ bytes,
                        const uint32_t *__restrict__ off, const uint32_t *__restrict__ by_len,
                        unsigned short *__restrict__ next, uint32_t *__restrict__ maskT,
                        unsigned lds, unsigned ldb, int row, int n_states, int n_classes, int V,
                        int eos_id, long long bytes_len, unsigned long long *oob)
{
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned short *s_tt = (unsigned short *)smem;            // [n_classes][compact_stride]
    uint8_t *s_cls = smem + (size_t)n_classes * compact_stride(n_states) * 2;   // [256]
    stage_compact_table(tt, row, n_states, n_classes, s_tt);
    for (int i = threadIdx.x; i < 256; i += blockDim.x)
        s_cls[i] = cls[i];
    __syncthreads();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const bool in = i < V;
    const unsigned v = in ? by_len[i] : 0u;
    const uint32_t b0 = in ? off[v] : 0u;
    int len = in ? (int)(off[v + 1] - b0) : 0;
    if (len > 0 && !CSTR_INB(oob, (long long)b0 + len - 1, bytes_len, CSTR_SITE_BUILD_VOCAB))
        len = 0;
    const bool is_eos = in && (int)v == eos_id;
    unsigned long long c_lo = 0ull, c_hi = 0ull;              // classes of bytes 0..7 and 8..15
    for (int k = 0; k < len && k < 16; ++k) {
        const unsigned long long c = (unsigned long long)s_cls[bytes[b0 + k]] << (8 * (k & 7));
        if (k < 8)
            c_lo |= c;
        else
            c_hi |= c;
    }
    const unsigned sink = (unsigned)n_states * 2u;
    const unsigned row_bytes = (unsigned)compact_stride(n_states) * 2u;
    const unsigned char *tb = (const unsigned char *)s_tt;
    uint32_t *mrow = maskT + (unsigned long long)v * ldb;
    const bool walks = in && len > 0 && !is_eos;
    uint32_t bits = 0u;
    for (int q0 = 0; q0 < n_states; q0 += 8) {
        unsigned cur[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
            cur[j] = (walks && q0 + j < n_states) ? (unsigned)(q0 + j) * 2u : sink;
        if (walks) {
            for (int k = 0; k < len; ++k) {
                const unsigned c = k < 16 ? (unsigned)((k < 8 ? c_lo : c_hi) >> (8 * (k & 7))) & 0xffu
                                          : (unsigned)s_cls[bytes[b0 + k]];
                const unsigned char *rowp = tb + c * row_bytes;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    cur[j] = *(const unsigned short *)(rowp + cur[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int q = q0 + j;
            const bool ok = is_eos ? (q < n_states && accept[q] != 0) : cur[j] != sink;
            bits |= (uint32_t)ok << (q & 31);
        }
        if (in && (((q0 + 8) & 31) == 0 || q0 + 8 >= n_states) &&
            CSTR_INB(oob, q0 >> 5, ldb, CSTR_SITE_BUILD_MASKT)) {   // a word of 32 states is complete
            mrow[q0 >> 5] = bits;
            bits = 0u;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            cur[j] = permuted_code(cur[j]);
        if (in && CSTR_INB(oob, q0 + 7, lds, CSTR_SITE_BUILD_NEXT))   // lds is a multiple of 256 entries
            *(uint4 *)(next + (unsigned long long)v * lds + q0) =
                make_uint4(cur[0] | (cur[1] << 16), cur[2] | (cur[3] << 16), cur[4] | (cur[5] << 16),
                           cur[6] | (cur[7] << 16));
    }
}

// ---- large automata: class rows staged by bulk copies --------------------------
//
// When the class-major table does not fit in shared memory (a random
// 10,000-state automaton with 256 byte classes: 5 MB), the walker above gathers
// 16-bit entries through L1 / L2, and the L1 tag stage becomes the bound.  One
// step of the walk, though, reads a single class row (S + 1 entries: 20 KB), and
// the sorted token list fixes the sequence of rows ahead of time.  So here ONE
// CTA covers all states (16 per lane), its warps take each step of the token
// sequence together, and a producer thread streams the rows of the coming
// steps into a ring in shared memory with bulk asynchronous copies
// (cp.async.bulk global -> shared, completion counted on an mbarrier); the
// lookups then are shared-memory loads.  Per ring slot a "full" barrier (the
// copy has landed) and an "empty" barrier (every consumer warp is done with
// it) hand the slot back and forth.  Every wait is bounded: a wait that runs
// out sets the CTA's abort flag and the table's status word, the consumers
// leave, and the producer waits for the copies it still has in flight.
constexpr int kRowsNS = 16;                  // states per lane
constexpr int kRowsMaxRing = 8;
constexpr int kRowsMinWarps = 18;            // below 18 x 512 states the L1 / L2 gather path is faster
constexpr unsigned kSpinLimit = 1u << 18;    // try_wait rounds before a wait gives up
constexpr unsigned kRowsHeader = 1280;       // row ids (1 KB), barriers (128 B), abort flag
constexpr int kRowsMaxThreads = 704;         // 21 consumer warps (10,752 states) + the producer warp

__device__ __forceinline__ unsigned smem_u32(const void *ptr)
{
    return (unsigned)__cvta_generic_to_shared(ptr);
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, unsigned count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t *bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0u;
}
// Bounded wait; false if it gave up (then the abort flag is set) or another warp did.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, unsigned parity, volatile int *abort_flag)
{
    for (unsigned round = 0; round < kSpinLimit; ++round) {
        if (mbar_try_wait(bar, parity))
            return true;
        if ((round & 255u) == 255u && *abort_flag)
            return false;
    }
    *abort_flag = 1;
    return false;
}
// This GPU's own global memory -> this CTA's shared memory, 16-byte aligned both, size a
// multiple of 16; completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_copy_g2s(void *dst_smem, const void *src, unsigned bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst_smem)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__global__ void __launch_bounds__(kRowsMaxThreads, 1)
build_rows_kernel(const __grid_constant__ BuildParams p, int n_cons, int ring, unsigned row_bytes,
                  unsigned *status)
{
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int NS = kRowsNS;
    uint32_t *s_cls = (uint32_t *)smem;                          // byte -> class row index
    uint64_t *full = (uint64_t *)(smem + 1024), *empty = full + kRowsMaxRing;
    volatile int *s_abort = (volatile int *)(smem + 1024 + 16 * kRowsMaxRing);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint4 *s_stack = (uint4 *)(smem + kRowsHeader);              // [depth][warp][lane][2]
    unsigned char *s_ring = smem + kRowsHeader + (size_t)(kDepth + 1) * n_cons * 32 * 32;

    for (int i = threadIdx.x; i < 256; i += blockDim.x)
        s_cls[i] = p.cls[i];
    if (threadIdx.x == 0) {
        for (int k = 0; k < ring; ++k) {
            mbar_init(full + k, 1u);
            mbar_init(empty + k, (unsigned)n_cons);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const int c_begin = blockIdx.x * p.tokens_per_cta;
    const int c_end = min(p.V, c_begin + p.tokens_per_cta);
    if (c_begin >= c_end)
        return;

    if (warp == n_cons) {
        // ---- producer: the rows of the step sequence, in order ----
        // The warp reads 32 descriptors at a time and works out each token's steps
        // in parallel; lane 0 then issues the copies token by token (the other
        // lanes only hand it their token's bytes), so that no global-memory
        // latency sits between two copies.
        unsigned issued = 0;
        int slot = 0;
        bool ok = true;
        for (int base = c_begin; base < c_end && ok; base += 32) {
            const int i = base + lane;
            const bool valid = i < c_end;
            uint4 d = make_uint4(0u, 0u, 0u, 0u);
            if (valid)
                d = __ldg(p.desc + i);
            const bool first = i == c_begin;
            const int n = (int)(d.y & 0xffffffu);
            const int sh = first ? 0 : (int)(d.y >> 24);
            const int m = valid ? n - sh : 0;
            uint32_t gb = 0u;
            if (m > 0 && (first || m > 8))
                gb = __ldg(p.off + d.x) + (uint32_t)sh;
            for (int t = 0; t < 32 && ok; ++t) {
                const int mt = __shfl_sync(kFull, m, t);
                if (mt == 0)
                    continue;                            // warp-uniform
                const unsigned z = __shfl_sync(kFull, d.z, t), w = __shfl_sync(kFull, d.w, t);
                const uint32_t gbt = __shfl_sync(kFull, gb, t);
                const bool inline_bytes = base + t != c_begin;
                if (lane == 0) {
                    for (int k = 0; k < mt; ++k) {
                        unsigned b;
                        if (inline_bytes && k < 8)
                            b = __byte_perm(z, w, (unsigned)k) & 0xffu;
                        else
                            b = __ldg(p.bytes + gbt + k);
                        if (issued >= (unsigned)ring &&
                            !mbar_wait(empty + slot, ((issued / (unsigned)ring) - 1u) & 1u, s_abort)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(full + slot, row_bytes);
                        // (class rows lie inside the table: (class + 1) * row_bytes <= tt_bytes)
                        const size_t src_off =
                            CSTR_INB(p.oob, ((long long)s_cls[b] + 1) * row_bytes - 1, p.tt_bytes,
                                     CSTR_SITE_BUILD_TT) ? (size_t)s_cls[b] * row_bytes : 0;
                        bulk_copy_g2s(s_ring + (size_t)slot * row_bytes,
                                      (const unsigned char *)p.tt + src_off, row_bytes, full + slot);
                        ++issued;
                        if (++slot == ring)
                            slot = 0;
                    }
                }
                ok = __shfl_sync(kFull, (int)ok, 0) != 0;
            }
        }
        if (lane != 0)
            return;
        if (!ok)
            atomicOr(status, 1u);
        // no copy may be in flight when the CTA's shared memory goes away
        const unsigned from = issued > (unsigned)ring ? issued - (unsigned)ring : 0u;
        for (unsigned t = from; t < issued; ++t) {
            uint64_t *bar = full + t % (unsigned)ring;
            const unsigned parity = (t / (unsigned)ring) & 1u;
            bool landed = false;
            for (unsigned round = 0; round < kSpinLimit && !landed; ++round)
                landed = mbar_try_wait(bar, parity);
            if (!landed)
                atomicOr(status, 2u);
        }
        return;
    }

    // ---- consumers: lane l of warp w holds states 512 w + 16 l .. + 15 ----
    const unsigned sink = (unsigned)CSTR_PERM(p.n_states) * 2u;
    const int q0 = warp * NS * 32, qbase = q0 + NS * lane;
    unsigned par[NS], cur[NS];
    unsigned accbits = 0;
#pragma unroll
    for (int j = 0; j < NS; ++j) {
        const bool in = qbase + j < p.n_states;
        accbits |= (unsigned)(in && p.accept[p.unrank ? p.unrank[qbase + j] : qbase + j] != 0) << j;
        par[j] = in ? (unsigned)CSTR_PERM(qbase + j) * 2u : sink;
        cur[j] = par[j];
    }
    const bool row_ok = qbase < (int)p.lds;              // the lane's 16 entries lie inside a token's row
    unsigned short *const next_lane = (unsigned short *)p.next + qbase;
    uint32_t *const maskT_warp = p.maskT + (q0 >> 5);
    uint4 *const my_stack = s_stack + ((size_t)warp * 32 + lane) * 2;
    const size_t level = (size_t)n_cons * 32 * 2;        // uint4 units per stack level

    auto pack2 = [&](const unsigned (&st)[NS], uint4 &a, uint4 &b) {
        a = make_uint4(st[0] | (st[1] << 16), st[2] | (st[3] << 16), st[4] | (st[5] << 16), st[6] | (st[7] << 16));
        b = make_uint4(st[8] | (st[9] << 16), st[10] | (st[11] << 16), st[12] | (st[13] << 16),
                       st[14] | (st[15] << 16));
    };
    auto push = [&](int depth, const unsigned (&st)[NS]) {
        uint4 a, b;
        pack2(st, a, b);
        my_stack[depth * level] = a;
        my_stack[depth * level + 1] = b;
    };
    auto pull = [&](int depth, unsigned (&st)[NS]) {
        const uint4 a = my_stack[depth * level], b = my_stack[depth * level + 1];
        const unsigned w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            st[2 * j] = w[j] & 0xffffu;
            st[2 * j + 1] = w[j] >> 16;
        }
    };
    push(0, par);
    __syncwarp();

    int slot = 0;
    unsigned phase = 0u;
    bool alive = true;                                   // false once a wait gave up
    // One step of the walk, taken by all consumer warps on the same staged row.
    auto step = [&](const unsigned (&src)[NS], unsigned (&dst)[NS]) {
        const bool ready = mbar_wait(full + slot, phase, s_abort);
        if (!__all_sync(kFull, ready)) {
            alive = false;
            return;
        }
        const unsigned char *rowp = s_ring + (size_t)slot * row_bytes;
#pragma unroll
        for (int j = 0; j < NS; ++j)
            dst[j] = CSTR_INB(p.oob, src[j], row_bytes, CSTR_SITE_BUILD_TT)
                         ? (unsigned)*(const unsigned short *)(rowp + src[j]) : sink;
        __syncwarp();                                    // every lane's loads of this slot are done
        if (lane == 0)
            mbar_arrive(empty + slot);
        if (++slot == ring) {
            slot = 0;
            phase ^= 1u;
        }
    };

    uint4 out_a, out_b;
    uint32_t words[NS];
    const uint4 dead_a = make_uint4(sink | (sink << 16), sink | (sink << 16), sink | (sink << 16),
                                    sink | (sink << 16));
    auto outputs_of = [&](const unsigned (&st)[NS]) {
        pack2(st, out_a, out_b);
#pragma unroll
        for (int j = 0; j < NS; ++j)
            words[j] = __ballot_sync(kFull, st[j] != sink);
    };
    auto store_outputs = [&](unsigned tok) {
        if (!CSTR_INB(p.oob, tok, p.V, CSTR_SITE_BUILD_NEXT) ||
            !CSTR_INB(p.oob, (q0 >> 5) + NS - 1, p.ldb, CSTR_SITE_BUILD_MASKT))
            return;
        if (row_ok) {
            uint4 *dst = (uint4 *)(next_lane + (unsigned long long)tok * p.lds);
            dst[0] = out_a;
            dst[1] = out_b;
        }
        if (lane == 0) {                 // 16 words of the token's ballot row, 64-byte aligned
            uint4 *mrow = (uint4 *)(maskT_warp + (unsigned long long)tok * p.ldb);
            mrow[0] = make_uint4(words[0], words[1], words[2], words[3]);
            mrow[1] = make_uint4(words[4], words[5], words[6], words[7]);
            mrow[2] = make_uint4(words[8], words[9], words[10], words[11]);
            mrow[3] = make_uint4(words[12], words[13], words[14], words[15]);
        }
    };

    // The same walk as build_trie_kernel: parent state in registers, stack levels
    // stored only while a later token can resume there, runs of repeated tokens
    // emitted at once.  The number of steps per token depends on the descriptors
    // alone, so producer and consumers agree on the sequence of rows.
    int pd = 0;
    bool first = true;
    uint4 d = __ldg(p.desc + c_begin);
#pragma unroll 1
    for (int i = c_begin; i < c_end && alive; ++i) {
        uint4 dn = make_uint4(0u, 0xffffffffu, 0u, 0u);
        int nsh = 0;
        if (i + 1 < c_end) {
            dn = __ldg(p.desc + i + 1);
            nsh = (int)(dn.y >> 24);
        }
        const unsigned tok = d.x;
        const int n = (int)(d.y & 0xffffffu);
        const int sh = first ? 0 : (int)(d.y >> 24);
        const bool is_eos = (int)tok == p.eos_id;
        if (sh != pd) {
            pull(sh, par);
            pd = sh;
        }
        const int m = n - sh;
        if (m == 0) {
            outputs_of(par);
        } else {
            step(par, cur);
#pragma unroll 1
            for (int k = 1; k < m && alive; ++k) {
                if (sh + k <= nsh)
                    push(sh + k, cur);
                step(cur, cur);
            }
            if (!alive)
                break;
            outputs_of(cur);
            if (n <= nsh) {
                push(n, cur);
#pragma unroll
                for (int j = 0; j < NS; ++j)
                    par[j] = cur[j];
                pd = n;
            }
        }
        if (n == 0 || is_eos) {
            out_a = out_b = dead_a;
#pragma unroll
            for (int j = 0; j < NS; ++j)
                words[j] = __ballot_sync(kFull, is_eos && ((accbits >> j) & 1u));
        }
        store_outputs(tok);
        first = false;
        if (!is_eos && n <= kDepth) {
            const unsigned same = (unsigned)n | ((unsigned)n << 24);
            while (dn.y == same && (int)dn.x != p.eos_id) {
                ++i;
                store_outputs(dn.x);
                dn = make_uint4(0u, 0xffffffffu, 0u, 0u);
                if (i + 1 < c_end)
                    dn = __ldg(p.desc + i + 1);
            }
        }
        d = dn;
    }
    if (!alive && lane == 0)
        atomicOr(status, 4u);
}

// ---- per-token walker without the trie ---------------------------------------
//
// Algorithm 1 taken literally: every token is its own chain of the detokenizing
// transducer, walked from its first byte for every state, with no prefix shared
// between tokens.  One thread per (state, token): a CTA holds 256 consecutive
// states of one token, looks the class-major table up through L1 / L2, stores
// its entry of the token's row and contributes its bit to the ballot word of
// its 32 states.  Kept as the baseline that shows what walking the trie-shaped
// T_V (Section 2.3) saves; cstr_table_build never takes this path.
template <typename ST, typename NT>
__global__ void __launch_bounds__(256)
build_dense_kernel(const __grid_constant__ BuildParams p)
{
    constexpr int ESZ = (int)sizeof(ST);
    typedef typename Unit<ESZ>::type SU;
    const unsigned v = blockIdx.x;
    const int q = blockIdx.y * 256 + threadIdx.x;
    const unsigned sink = (unsigned)CSTR_PERM(p.n_states) * ESZ;
    const bool in = q < p.n_states;
    unsigned cur = in ? (unsigned)CSTR_PERM(q) * ESZ : sink;
    const uint32_t b0 = __ldg(p.off + v), n = __ldg(p.off + v + 1) - b0;
    const bool is_eos = (int)v == p.eos_id;
    const unsigned char *g_tt = (const unsigned char *)p.tt;
    bool ok;
    if (is_eos || n == 0) {
        ok = is_eos && in && p.accept[p.unrank ? p.unrank[q] : q] != 0;
        cur = sink;
    } else {
        for (uint32_t k = 0; k < n; ++k) {
            if (!CSTR_INB(p.oob, (long long)b0 + k, p.bytes_len, CSTR_SITE_BUILD_VOCAB))
                break;
            const unsigned c = __ldg(p.cls + __ldg(p.bytes + b0 + k));
            if (!CSTR_INB(p.oob, (long long)c * p.row * ESZ + cur, p.tt_bytes, CSTR_SITE_BUILD_TT)) {
                cur = sink;
                break;
            }
            cur = (unsigned)__ldg((const SU *)(g_tt + (size_t)c * p.row * ESZ + cur));
        }
        ok = cur != sink;
    }
    if (CSTR_INB(p.oob, q, p.lds, CSTR_SITE_BUILD_NEXT))
        ((NT *)p.next)[(unsigned long long)v * p.lds + q] = (NT)cur;   // q < lds (a multiple of 256)
    const unsigned word = __ballot_sync(kFull, ok);
    if ((threadIdx.x & 31) == 0 && CSTR_INB(p.oob, q >> 5, p.ldb, CSTR_SITE_BUILD_MASKT))
        p.maskT[(unsigned long long)v * p.ldb + (q >> 5)] = word;      // word k: states 32 k .. 32 k + 31
}

template <typename ST, typename NT, int NS, bool SMEM, bool PRUNE>
cudaError_t launch_trie(const BuildParams &p, dim3 grid, int threads, size_t smem_bytes,
                        cudaStream_t stream)
{
    auto kernel = build_trie_kernel<ST, NT, NS, SMEM, PRUNE>;
    if (smem_bytes > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem_bytes);
        if (e != cudaSuccess)
            return e;
    }
    kernel<<<grid, threads, smem_bytes, stream>>>(p);
    return cudaGetLastError();
}

template <typename ST, typename NT>
cudaError_t launch_trie_ns(int ns, bool in_smem, bool prune, const BuildParams &p, dim3 grid,
                           int threads, size_t smem_bytes, cudaStream_t stream)
{
#define CSTR_CASE(N)                                                                               \
    return in_smem ? (prune ? launch_trie<ST, NT, N, true, true>(p, grid, threads, smem_bytes, stream)    \
                            : launch_trie<ST, NT, N, true, false>(p, grid, threads, smem_bytes, stream))  \
                   : (prune ? launch_trie<ST, NT, N, false, true>(p, grid, threads, smem_bytes, stream)   \
                            : launch_trie<ST, NT, N, false, false>(p, grid, threads, smem_bytes, stream))
    switch (ns) {
    case 1: CSTR_CASE(1);
    case 2: CSTR_CASE(2);
    case 4: CSTR_CASE(4);
    default:
        if constexpr (sizeof(NT) == 2) {
            CSTR_CASE(8);
        } else {
            CSTR_CASE(4);
        }
    }
#undef CSTR_CASE
}

}  // namespace

#ifdef CSTR_TESTING
extern "C" int cstr_test_set_group_hash_bits(int32_t bits)
{
    if (bits < 0 || bits > 64)
        return cstr_fail(CSTR_ERR_ARG, "cstr_test_set_group_hash_bits: bits = %d, need 0..64", bits);
    g_test_hash_keep = (bits == 0 || bits == 64) ? ~0ull : (1ull << bits) - 1ull;
    return CSTR_OK;
}
#endif

// Post-pass for automata with terminal-label edges (no-op otherwise).
static int launch_terminals(cstr_table *t, const cstr_dfa *dfa, cudaStream_t stream)
{
    const cstr_vocab *vc = t->vocab;
    const int S = dfa->n_states;
    if (dfa->n_term_states > 0) {
        const unsigned sink = (unsigned)CSTR_PERM(S) << (dfa->wide ? 2 : 1);
        const unsigned agrid = (unsigned)((t->V + 255) / 256);
        if (t->wide)
            apply_terminals_kernel<uint32_t><<<agrid, 256, 0, stream>>>(
                dfa->tstate, dfa->tset, dfa->ttarget, dfa->n_term_states, dfa->n_labels, vc->tsets,
                vc->off, t->V, t->eos_id, sink, dfa->rank, (uint32_t *)t->next, t->lds, t->mask,
                t->ldw, (long long)t->max_states * t->ldw, CSTR_OOB_RECORD());
        else
            apply_terminals_kernel<uint16_t><<<agrid, 256, 0, stream>>>(
                dfa->tstate, dfa->tset, dfa->ttarget, dfa->n_term_states, dfa->n_labels, vc->tsets,
                vc->off, t->V, t->eos_id, sink & 0xffffu, dfa->rank, (uint16_t *)t->next, t->lds,
                t->mask, t->ldw, (long long)t->max_states * t->ldw, CSTR_OOB_RECORD());
        CSTR_CUDA_TRY(cudaGetLastError());
    }
    return CSTR_OK;
}

int cstr_launch_build(cstr_table *t, const cstr_dfa *dfa, cudaStream_t stream, bool dense_walk)
{
    const cstr_vocab *vc = t->vocab;
    BuildParams p;
    p.tt = dfa->tt;
    p.cls = dfa->cls;
    p.accept = dfa->accept;
    p.unrank = dfa->unrank;
    p.desc = vc->desc;
    p.pre4 = vc->pre4;
    p.bytes = vc->bytes;
    p.off = vc->off;
    p.next = t->next;
    p.maskT = t->maskT;
    p.row = (int)dfa->row;
    p.lds = (unsigned)t->lds;      // at most 4,000,512 states
    p.ldb = (unsigned)t->ldb;
    p.n_states = dfa->n_states;
    p.n_classes = dfa->n_classes;
    p.V = t->V;
    p.eos_id = t->eos_id;
    p.oob = CSTR_OOB_RECORD();
    p.tt_bytes = (long long)dfa->n_classes * dfa->row * (dfa->wide ? 4 : 2);
    p.bytes_len = vc->total_bytes + 16;
    p.mask_words = (long long)t->max_states * t->ldw;
    MetaCopy meta;
    meta.accept_src = dfa->accept;
    meta.accept_dst = t->accept;
    meta.n_states = dfa->n_states;
    meta.rank_src = dfa->rank;
    meta.rank_dst = t->rank;
    meta.rank_words = dfa->rank ? 2 * (dfa->n_states + 1) : 0;

    if (dfa->wide && !t->wide)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_table_build: DFA wider than the table");
    const size_t st = dfa->wide ? 4 : 2;

    if (dense_walk) {                  // the baseline walker: every token from its first byte
        p.count_dev = nullptr;
        p.reptok = nullptr;
        dim3 grid((unsigned)t->V, (unsigned)((dfa->n_states + 255) / 256));
        if (!dfa->wide && !t->wide)
            build_dense_kernel<int16_t, int16_t><<<grid, 256, 0, stream>>>(p);
        else if (!dfa->wide && t->wide)
            build_dense_kernel<int16_t, int32_t><<<grid, 256, 0, stream>>>(p);
        else
            build_dense_kernel<int32_t, int32_t><<<grid, 256, 0, stream>>>(p);
        CSTR_CUDA_TRY(cudaGetLastError());
        const int words = (dfa->n_states + 31) / 32;
        dim3 tg((unsigned)(t->ldw / 32), (unsigned)((words + 7) / 8));
        mask_transpose_kernel<<<tg, 256, 0, stream>>>(t->maskT, t->ldb, t->mask, t->ldw,
                                                      dfa->n_states, t->V, 1, nullptr, dfa->unrank,
                                                      p.mask_words, p.oob, meta);
        CSTR_CUDA_TRY(cudaGetLastError());
        return launch_terminals(t, dfa, stream);
    }

    // Small automata: one lane per token, all states in turn, mask words by ballot.
    const size_t small_smem =          // at most 256 x 66 x 2 + 256 bytes
        dfa->n_states <= kLaneTokenStates
            ? (size_t)dfa->n_classes * (size_t)compact_stride(dfa->n_states) * 2 + 256 : 0;
    if (!dfa->wide && !t->wide && dfa->n_states <= kSmallStates) {
        const int warps = 8;
        build_small_kernel<<<(unsigned)((t->W + warps - 1) / warps), warps * 32, small_smem, stream>>>(
            (const unsigned short *)dfa->tt, dfa->cls, dfa->accept, vc->bytes, vc->off,
            (unsigned short *)t->next, t->mask, (unsigned)t->lds, t->ldw, (int)dfa->row,
            dfa->n_states, dfa->n_classes, t->V, t->W, t->eos_id, p.bytes_len, p.oob);
        CSTR_CUDA_TRY(cudaGetLastError());
        table_meta_kernel<<<1, 256, 0, stream>>>(meta);          // no transpose pass on this path
        CSTR_CUDA_TRY(cudaGetLastError());
        return launch_terminals(t, dfa, stream);
    }

    // A little larger: lane = token over tokens of equal length, then the transpose pass.
    const int lane_token_states = kLaneTokenStates;
    const size_t lt_smem = small_smem;
    if (!dfa->wide && !t->wide && dfa->n_states <= lane_token_states) {
        build_lane_token_kernel<<<(unsigned)((t->V + 255) / 256), 256, lt_smem, stream>>>(
            (const unsigned short *)dfa->tt, dfa->cls, dfa->accept, vc->bytes, vc->off, vc->by_len,
            (unsigned short *)t->next, t->maskT, (unsigned)t->lds, (unsigned)t->ldb, (int)dfa->row,
            dfa->n_states, dfa->n_classes, t->V, t->eos_id, p.bytes_len, p.oob);
        CSTR_CUDA_TRY(cudaGetLastError());
        const int words = (dfa->n_states + 31) / 32;
        dim3 tg((unsigned)(t->ldw / 32), (unsigned)((words + 7) / 8));
        mask_transpose_kernel<<<tg, 256, 0, stream>>>(t->maskT, t->ldb, t->mask, t->ldw,
                                                      dfa->n_states, t->V, 1, nullptr, nullptr,
                                                      p.mask_words, p.oob, meta);
        CSTR_CUDA_TRY(cudaGetLastError());
        return launch_terminals(t, dfa, stream);
    }

    // Duplicate-column pass for large automata with few byte classes over a large
    // vocabulary (elsewhere class strings rarely repeat, or the walk is too short
    // for the extra passes to pay).
    const bool dedup = dfa->n_classes <= kDedupMaxClasses && t->V >= kDedupMinTokens &&
                       dfa->n_states >= kDedupMinStates;
    p.count_dev = nullptr;
    p.reptok = nullptr;
    if (dedup) {
        CSTR_CUDA_TRY(cudaMemsetAsync(t->group_key, 0, (size_t)t->group_slots * 8, stream));
        CSTR_CUDA_TRY(cudaMemsetAsync(t->group_min, 0xff, (size_t)t->group_slots * 4, stream));
        const unsigned g = (unsigned)((t->V + 255) / 256);
        unsigned long long keep = ~0ull;
#ifdef CSTR_TESTING
        keep = g_test_hash_keep;     // checking build only: fewer hash bits force collisions
#endif
        // A small first launch seeds the table: thousands of tokens share a few
        // popular class strings, and once a group's minimum is in place the bulk
        // of the tokens finds it with plain loads instead of same-address atomics.
        const int seed = 4096;
        group_insert_kernel<<<seed / 256, 256, 0, stream>>>(vc->desc, vc->bytes, vc->off, dfa->cls, 0,
                                                            seed, t->eos_id, t->group_key,
                                                            t->group_min, t->group_slots, keep);
        group_insert_kernel<<<(unsigned)((t->V - seed + 255) / 256), 256, 0, stream>>>(
            vc->desc, vc->bytes, vc->off, dfa->cls, seed, t->V, t->eos_id, t->group_key,
            t->group_min, t->group_slots, keep);
        const int n_blk = (t->V + 1023) / 1024;
        group_resolve_kernel<<<n_blk, 1024, 0, stream>>>(vc->desc, vc->bytes, vc->off, dfa->cls, t->V,
                                                         t->eos_id, t->group_key, t->group_min,
                                                         t->group_slots, keep, t->group_rep,
                                                         t->group_reptok, t->group_blk);
        group_scan_kernel<<<1, 1024, 0, stream>>>(t->group_blk, n_blk, t->group_count);
        group_scatter_kernel<<<n_blk, 1024, 0, stream>>>(t->group_rep, t->V, t->group_blk,
                                                         t->group_uniq);
        group_desc_kernel<<<g, 256, 0, stream>>>(vc->desc, t->group_uniq, t->group_count, vc->bytes,
                                                 vc->off, t->group_desc);
        CSTR_CUDA_TRY(cudaGetLastError());
        p.desc = t->group_desc;
        p.pre4 = nullptr;            // the representatives' own list has no such array
        p.count_dev = t->group_count;
        p.reptok = t->group_reptok;
    }

    // Large automata whose table cannot sit in shared memory: one CTA over all states,
    // class rows staged by bulk copies (build_rows_kernel).
    {
        const size_t row_bytes = (size_t)dfa->row * 2;
        const int n_cons = (dfa->n_states + kRowsNS * 32 - 1) / (kRowsNS * 32);
        const size_t stack_bytes = (size_t)(kDepth + 1) * n_cons * 32 * 32;
        const size_t smem_max = 227 * 1024;
        const size_t table_bytes_all = (size_t)dfa->n_classes * row_bytes;
        long long ring = smem_max > kRowsHeader + stack_bytes
                             ? (long long)((smem_max - kRowsHeader - stack_bytes) / row_bytes) : 0;
        if (ring > kRowsMaxRing)
            ring = kRowsMaxRing;
        // a second CTA on the SM (small automata) is worth more than a deep ring
        while (ring > 4 && 2 * (kRowsHeader + stack_bytes + (size_t)ring * row_bytes) > smem_max &&
               2 * (kRowsHeader + stack_bytes + 4 * row_bytes) <= smem_max)
            --ring;
        // Measured against the gather path on random automata with 256 byte classes over
        // 256,000 tokens: slower below about 9,000 states (2,048: 0.80 vs 0.57 ms; 6,144:
        // 2.05 vs 1.79; 8,192: 2.26 vs 2.20), faster above (10,000: 2.47 vs 2.85 ms).
        if (!dedup && !dfa->wide && !t->wide && !dfa->sparse && table_bytes_all > 190 * 1024 &&
            n_cons >= kRowsMinWarps && (n_cons + 1) * 32 <= kRowsMaxThreads && ring >= 3) {
            int dev_sms = 148;
            cudaDeviceGetAttribute(&dev_sms, cudaDevAttrMultiProcessorCount, t->device);
            long long chunks = 4LL * dev_sms;
            long long per = (t->V + chunks - 1) / chunks;
            if (per < 64)
                per = 64;
            chunks = (t->V + per - 1) / per;
            p.tokens_per_cta = (int)per;
            p.count_dev = nullptr;
            p.reptok = nullptr;
            const size_t smem_bytes = kRowsHeader + stack_bytes + (size_t)ring * row_bytes;
            CSTR_CUDA_TRY(cudaFuncSetAttribute(build_rows_kernel,
                                               cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               (int)smem_bytes));
            build_rows_kernel<<<(unsigned)chunks, (n_cons + 1) * 32, smem_bytes, stream>>>(
                p, n_cons, (int)ring, (unsigned)row_bytes, t->build_status);
            CSTR_CUDA_TRY(cudaGetLastError());
            const int words = n_cons * kRowsNS;
            dim3 tg((unsigned)(t->ldw / 32), (unsigned)((words + 7) / 8));
            mask_transpose_kernel<<<tg, 256, 0, stream>>>(t->maskT, t->ldb, t->mask, t->ldw,
                                                          dfa->n_states, t->V, kRowsNS, nullptr,
                                                          dfa->unrank, p.mask_words, p.oob, meta);
            CSTR_CUDA_TRY(cudaGetLastError());
            return launch_terminals(t, dfa, stream);
        }
    }

    // States per lane: enough states per warp to amortise the per-token work,
    // without leaving most lanes idle on small automata.
    const int S = dfa->n_states;
    // A warp's cost per token is mostly fixed (about 116 instructions measured)
    // plus about 4.3 per state held by a lane, so take the NS with the fewest
    // instructions over all state blocks.  (16 states per lane was tried: fewer
    // instructions still, but too few resident warps to hide the latencies.)
    int ns = 1;
    long long best_cost = -1;
    for (int cand = 1; cand <= (t->wide ? 4 : 8); cand *= 2) {   // a lane's unit of next is <= 16 bytes
        const long long blocks = (S + 32 * cand - 1) / (32 * cand);
        const long long cost = blocks * (1160 + 43 * cand);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost;
            ns = cand;
        }
    }
    const int per_warp = ns * 32;
    const int state_warps = (S + per_warp - 1) / per_warp;

    // Warps per CTA from the shared-memory budget: the table (when it fits) is
    // shared by all warps of a CTA, each warp adds its per-depth stack.  Aim
    // for two resident CTAs per SM, fall back to one big CTA for large tables.
    const size_t stack_per_warp = (size_t)(CSTR_STACK_DEPTH + 1) * ns * 32 * st;
    const size_t table_bytes = (size_t)dfa->n_classes * (size_t)dfa->row * st;
    const size_t cta_max = 200 * 1024, cta_half = 108 * 1024;
    const bool in_smem = 1024 + 4 * stack_per_warp + table_bytes <= cta_max;
    const size_t fixed = 1024 + (in_smem ? table_bytes : 0);
    size_t budget = in_smem ? cta_half : 48 * 1024;
    int warp_cap = 16;
    bool one_cta_per_sm = false;
    if (fixed + 8 * stack_per_warp > budget) {
        budget = cta_max;            // one CTA per SM: let it hold all the warps the register
        one_cta_per_sm = true;       // file allows (the 8-states-per-lane kernels fit 1,024 threads)
        if (ns == 8)
            warp_cap = 32;
    }
    int max_warps = (int)((budget - fixed) / stack_per_warp);
    if (max_warps > warp_cap)
        max_warps = warp_cap;
    if (max_warps < 1)
        max_warps = 1;
    int state_groups = (state_warps + max_warps - 1) / max_warps;
    const int warps_s = (state_warps + state_groups - 1) / state_groups;   // balanced groups
    state_groups = (state_warps + warps_s - 1) / warps_s;
    int warps_t = max_warps / warps_s;
    if (warps_t < 1)
        warps_t = 1;
    const int warps = warps_s * warps_t;
    const int threads = warps * 32;
    const size_t smem_bytes = fixed + (size_t)warps * stack_per_warp;
    p.warps_s = warps_s;
    p.warps_t = warps_t;

    // Token chunks: every warp restarts its walk at the root of the trie, so a
    // warp's share should be long; but there must be enough CTAs for the machine.
    int dev_sms = 148;
    cudaDeviceGetAttribute(&dev_sms, cudaDevAttrMultiProcessorCount, t->device);
    const long long want_ctas = (table_bytes <= 16 * 1024 && in_smem ? 32LL : 8LL) * dev_sms;
    long long chunks = (want_ctas + state_groups - 1) / state_groups;
    long long tokens_per_cta = (t->V + chunks - 1) / chunks;
    // (a CTA re-stages the table, so big tables want long chunks; small automata
    // are latency-bound per token and want many short ones)
    const long long min_tokens =
        (long long)warps_t * (!in_smem ? 128 : (table_bytes <= 16 * 1024 ? 32 : 256));
    if (tokens_per_cta < min_tokens)
        tokens_per_cta = min_tokens;
    chunks = (t->V + tokens_per_cta - 1) / tokens_per_cta;
    if (one_cta_per_sm && state_groups * chunks < dev_sms) {
        // fewer CTAs than SMs and only one fits an SM: shorter chunks (at least
        // 32 tokens per warp) so that every SM gets one
        const long long fill = (dev_sms + state_groups - 1) / state_groups;
        const long long per = (t->V + fill - 1) / fill;
        tokens_per_cta = per > 32LL * warps_t ? per : 32LL * warps_t;
        chunks = (t->V + tokens_per_cta - 1) / tokens_per_cta;
    }
    if (chunks > 65535) {
        chunks = 65535;
        tokens_per_cta = (t->V + chunks - 1) / chunks;
        chunks = (t->V + tokens_per_cta - 1) / tokens_per_cta;
    }
    p.tokens_per_cta = (int)tokens_per_cta;
    // pruning walks: about four units per warp, so that the counter can even out
    // state blocks that die early against those that do not
    p.slice_tokens = (int)((tokens_per_cta + 4LL * warps_t - 1) / (4LL * warps_t));
    if (p.slice_tokens < 16)
        p.slice_tokens = 16;
    dim3 grid((unsigned)state_groups, (unsigned)chunks);

    // Sparse automata (most states allow few bytes): prune dead subtrees per warp.
    const bool prune = dfa->sparse != 0;
    cudaError_t e;
    if (!dfa->wide && !t->wide)
        e = launch_trie_ns<int16_t, int16_t>(ns, in_smem, prune, p, grid, threads, smem_bytes, stream);
    else if (!dfa->wide && t->wide)
        e = launch_trie_ns<int16_t, int32_t>(ns, in_smem, prune, p, grid, threads, smem_bytes, stream);
    else
        e = launch_trie_ns<int32_t, int32_t>(ns, in_smem, prune, p, grid, threads, smem_bytes, stream);
    if (e != cudaSuccess)
        return cstr_fail(CSTR_ERR_CUDA, "cstr_table_build: builder launch: %s",
                         cudaGetErrorString(e));

    const int ballot_words = ((S + per_warp - 1) / per_warp) * ns;
    if (dedup) {
        const size_t nt = t->wide ? 4 : 2;
        long long used = (long long)state_warps * per_warp;          // entries the walk wrote
        if (used > t->lds)
            used = t->lds;
        expand_rows_kernel<<<(unsigned)t->V, 256, 0, stream>>>(
            t->group_reptok, (unsigned char *)t->next, (unsigned long long)t->lds * nt,
            (int)(used * nt / 16), t->V, p.oob);
        CSTR_CUDA_TRY(cudaGetLastError());
    }
    dim3 tgrid((unsigned)(t->ldw / 32), (unsigned)((ballot_words + 7) / 8));
    if (tgrid.y > 65535u)
        return cstr_fail(CSTR_ERR_SHAPE, "cstr_table_build: too many states for one launch");
    mask_transpose_kernel<<<tgrid, 256, 0, stream>>>(t->maskT, t->ldb, t->mask, t->ldw, S, t->V,
                                                     ns, p.reptok, dfa->unrank, p.mask_words, p.oob, meta);
    CSTR_CUDA_TRY(cudaGetLastError());

    return launch_terminals(t, dfa, stream);
}
