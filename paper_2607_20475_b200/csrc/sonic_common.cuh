// Shared device-side definitions of the sonic kernels (sm_100a).
//
// Vocabulary layout: a row is cut into CTA tiles of 8192 elements (eight warp
// tiles of 1024); a lane owns 32 elements of its warp tile as 128-bit vectors,
// vector j of lane l starting at element j*32*VEC + l*VEC (fully coalesced).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <math_constants.h>

namespace sonic {

// mode bits (Section 3.5, indicator table)
constexpr uint32_t M_GRAMMAR = 0x001, M_REPETITION = 0x002, M_FREQUENCY = 0x004, M_PRESENCE = 0x008,
                   M_BIAS = 0x010, M_TEMPERATURE = 0x020, M_GREEDY = 0x040, M_TOP_K = 0x080,
                   M_TOP_P = 0x100, M_MIN_P = 0x200;
constexpr uint32_t M_PENALTIES = M_REPETITION | M_FREQUENCY | M_PRESENCE;

constexpr uint32_t F_NO_TOKEN = 0x1, F_BADPARAM = 0x2, F_FALLBACK = 0x4, F_DENSE = 0x8, F_TIMEOUT = 0x10;
constexpr uint32_t F_ACCEPT = 0x100;          // workspace only (per-position verification result)

constexpr int OP_SAMPLE = 0, OP_VERIFY = 1, OP_TOPK = 2;

constexpr int WARP_TILE = 1024;               // elements per warp tile
constexpr int EPL = 32;                       // elements per lane per warp tile
constexpr int STREAM_THREADS = 256;
constexpr int STREAM_WARPS = STREAM_THREADS / 32;
constexpr int CTA_TILE = WARP_TILE * STREAM_WARPS;   // 8192
constexpr int MAX_TILES = (262144 + CTA_TILE - 1) / CTA_TILE;   // 32 tiles at the largest vocabulary
// Sparse lists in the stream kernel: the producer warp keeps a request's lists in registers (up to FILTER_HIST
// history entries, id and count packed in one word, and FILTER_BIAS bias entries) and hands each tile the
// entries that fall into it; longer lists are scanned by the consumer threads.
constexpr int FILTER_HIST = 512;
constexpr int FILTER_BIAS = 32;
constexpr int FILTER_COUNT_MAX = (1 << 14) - 1;   // largest count that packs beside an 18-bit id
constexpr int HIT_PEN_CAP = 320;              // history entries of one tile the producer can hand over
constexpr int HIT_BIAS_CAP = FILTER_BIAS;
constexpr uint32_t CAND_CAP = 32768;          // candidate slots per row, divided evenly among the row's tiles
constexpr int MERGE_THREADS = 512;
constexpr int MERGE_CAP = 8192;               // 64-bit keys the row merge can sort (64 KB of shared memory)
constexpr int KFAST_SAMPLE = MERGE_CAP / 4;   // largest top-k the streaming path finishes for sampling rows (2048)
constexpr int KFAST_TOPK = MERGE_CAP / 2;     // ... and for sonic_topk rows (4096)
constexpr int MAX_TOPK = 4096;                // largest k of sonic_topk
constexpr int MAX_VOCAB = 262144;

constexpr int CLS_GREEDY = 0;                 // streaming path, argmax only
constexpr int CLS_TOPK = 1;                   // streaming path, candidates + merge
constexpr int CLS_EXACT = 2;                  // cluster kernel only (top-k beyond what the streaming path sorts)
constexpr int CLS_DENSE = 3;                  // top-k off: streaming pass for the keys, then the histogram passes

// Workspace header (the first WS_HEADER_WORDS 32-bit words; the only part of the workspace that must be zero
// between calls: every other word is initialised by the call that reads it)
constexpr int WS_ERROR = 0;                    // sticky ERR_* bits
constexpr int WS_FAILED_ROWS = 1;              // rows of the current call that the streaming or histogram path handed to the cluster kernel
constexpr int WS_QUEUE = 2;                    // the stream kernel's work counter
constexpr int WS_EXACT_TICKET = 3;             // next row ordinal of the cluster kernel
constexpr int WS_NDENSE = 4;                   // rows of the current call on the histogram path (length of the dense list)
constexpr int WS_NRESID = 5;                   // verification rows of the current call whose draft was rejected (length of the residual list)
constexpr int WS_EXACT_LEFT = 6;               // clusters of the cluster kernel that have run out of rows
constexpr int WS_NEXACT = 7;                   // rows of the current call that belong to the cluster kernel by class
constexpr int WS_TEST_WITHHOLD = 100;          // test-only builds (SONIC_TEST_WITHHOLD): 1 + the work item whose tile copy is withheld
constexpr int WS_HEADER_WORDS = 128;
constexpr uint32_t ST_FAILED = 0x1;           // streaming / histogram path could not finish the row
constexpr unsigned int ERR_TIMEOUT = 0x1;     // workspace header: a bounded mbarrier wait expired
constexpr uint32_t TILE_BADID = 0x1;          // TileRec.flags: a list id of the row was out of range

constexpr uint32_t KEY_NEG_INF = 0x007FFFFFu; // okey(-inf)

struct __align__(16) RowState {
    unsigned int status;                      // ST_*; set to zero by the streaming kernel, ST_FAILED by a row's finisher
    unsigned int pad[3];
};

struct __align__(16) TileRec {                // written by the tile's CTA in the streaming kernel
    unsigned long long best;                  // greedy and dense rows: largest (key << 32 | ~index) of the tile, 0 if none finite
    unsigned int cnt;                         // top-k rows: candidates of the tile (may exceed the slot: overflow)
    unsigned int tkey;                        // top-k rows: the tile's cutoff as an ordered key
    unsigned int minkey;                      // dense rows: smallest finite key of the tile (0xFFFFFFFF if none)
    unsigned int nfin;                        // dense rows: finite elements of the tile
    unsigned int flags;                       // TILE_*
    unsigned int pad;
};

// Histogram path (rows with top-k off), per row.  Initialised by the streaming kernel (the CTA of the row's first
// tile); the later passes communicate through it.
constexpr int DBINS = 2048;                   // bins of the mass histogram, uniform in (M - y)
constexpr int MEMBER_CAP = 4096;              // elements of the crossing bin that can be listed
struct __align__(16) DenseRow {
    unsigned int ticket_h, ticket_c, ticket_r, nmembers;     // items that have finished a pass; listed members
    unsigned int kmin, kmax, overflow, state;                // key span of the members; an item could not stage its members; 1 = collect pass wanted
    unsigned int Mkey, tk, klo, khi;                         // row maximum; min-p key threshold (0 = none); keys of the crossing bin: klo .. khi (empty if klo > khi)
    unsigned long long target;                               // mass the ranking prefix must reach (0: top-p does not decide inside the bin)
    unsigned long long cutc, W;                              // final cut (composite key) and total fixed-point mass of the support
    float p_draft; int support;
    unsigned int pad[4];
};
static_assert(sizeof(DenseRow) == 96, "DenseRow layout");
constexpr int DENSE_CHUNK = 512;                 // elements per chunk of a tile
constexpr int DENSE_CHUNKS = 16;                 // chunks per tile
struct __align__(16) DenseChunk {             // per chunk of 512 elements, written by pass C
    unsigned long long A;                     // fixed-point mass of the chunk's elements above the crossing bin
    unsigned int n, nb;                       // their number; the chunk's elements inside the crossing bin
};
struct __align__(16) DenseTile {              // per (row, tile) of the histogram path
    DenseChunk ch[DENSE_CHUNKS];
    unsigned long long mass;                  // fixed-point mass of the tile's part of the final support
    double R, Pp, S;                          // residual pass: sum of max(0, w/W~ - q), sum of w where that is positive, sum of w
};
static_assert(sizeof(DenseTile) == 288, "DenseTile layout");

struct __align__(16) PosResult {              // per logit row, verification only
    int token;
    unsigned int flags;                       // F_* | F_ACCEPT
    float p;                                  // p_l(d_l)
    int support;
};

struct KParams {
    int op, rows, V, K, ktop, dtype;
    const void *logits;
    long long row_stride;
    const uint32_t *mode;
    const uint32_t *bitmask;
    long long bitmask_stride;
    const float *temperature;
    const int *top_k;
    const float *top_p;
    const float *min_p;
    const float *rep, *freq, *pres;
    const int *hist_ids, *hist_counts, *hist_len;
    int hist_stride;
    const int *bias_ids;
    const float *bias_vals;
    const int *bias_len;
    int bias_stride;
    const unsigned long long *seed, *offset;
    const int *draft_tokens;
    const float *draft_probs;
    int *out_token;
    float *out_prob;
    uint32_t *out_flags;
    int *out_support;
    int *out_tokens;
    int *out_accept;
    float *out_pdraft;
    float *out_vals;
    int *out_idx;
    unsigned int *error;                      // workspace header (WS_* words); word 0: ERR_* (sticky)
    RowState *rs;
    TileRec *tiles;
    PosResult *pr;
    unsigned long long *cand;                 // [rows][cand_stride] candidate slots, split evenly among a row's tiles
    unsigned int cand_stride;
    // histogram path (sample / verify calls only)
    DenseRow *drow;                           // [rows]
    DenseTile *dtile;                         // [rows][MAX_TILES]
    int *dlist, *rlist;                       // [rows] rows on the histogram path; rows whose draft was rejected
    unsigned long long *hist;                 // [rows][DBINS] fixed-point mass per bin
    unsigned long long *members;              // [rows][MEMBER_CAP] elements of the crossing bin (key << 32 | ~index)
    unsigned int *ykeys;                      // [rows][ytiles * CTA_TILE] ordered keys of the processed logits
    int ytiles;
};

// Per-row configuration derived from the request's mode bits and parameters.
struct RowCfg {
    uint32_t z;
    int b, l;              // request, position within the request (0 outside verification)
    int k;                 // top-k bound, 0 = off
    float tau, p, theta;
    float alpha, beta, gamma;
    int hist_len, bias_len;
    int cls, G;            // path class; groups per warp tile (0 = keep every finite element)
    bool tile_min;         // the tile cutoff is the smallest warp cutoff (tile mode of pick_groups), not the largest
    bool bad;              // parameter outside its domain
    bool temp;             // temperature bit
    bool div_all;          // streaming path divides every element (greedy with temperature)
};

// Ordered key of a float: unsigned order == float order, -0 folded into +0.
__device__ __forceinline__ uint32_t okey(float f) {
    uint32_t b = __float_as_uint(__fadd_rn(f, 0.0f));
    return b ^ ((b & 0x80000000u) ? 0xFFFFFFFFu : 0x80000000u);
}
__device__ __forceinline__ float unkey(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}

// z / tau in IEEE round-to-nearest for a finite tau > 0.  Infinities and NaN (masked or padded entries) pass through
// unchanged without entering the division's slow path, which the whole warp would otherwise wait for.
__device__ __forceinline__ float div_tau(float z, float tau) {
    const bool special = !(fabsf(z) < CUDART_INF_F);
    const float q = __fdiv_rn(special ? 1.0f : z, tau);
    return special ? z : q;
}

// Which group maxima bound a tile's cutoff.  A warp tile (1024 elements) is cut into G groups (a power of
// two, 1..32, or 64 with half-lane groups) and the cutoff of a block is the smallest of its group maxima, so
// at least one element per group lies at or above it.  Two kinds of block:
//   warp mode: block = warp tile (G groups); the tile cutoff is the LARGEST of its eight warp cutoffs;
//   tile mode: block = the whole 8192-element tile (8 G groups); the tile cutoff is the SMALLEST warp cutoff.
// The row-wide cutoff T is the largest tile cutoff either way.  For position-independent data a block of m
// groups has a cutoff above t with probability (1 - exp(-x))^m, x = (elements above t per group), so with
// Nb blocks in the row T sits where 1 - exp(-x) = Nb^(-1/m), and the proven prefix holds about
//     P = V * (G / 1024) * -ln(1 - Nb^(-1/m))
// elements.  A minimum over more groups concentrates better: at V = 2^18 tile mode with G = 1 proves
// 245 elements on average (94 at worst in 400 simulated rows) where warp mode with G = 4 proves 265 (63 at
// worst) and G = 8 proves 1330.  The candidates are tried in the order of their P (warp 2, tile 1, warp 4,
// tile 2, warp 8, tile 4, warp 16, tile 8, warp 32, warp 64) and the first one is taken whose P clears k
// with a margin that covers the spread of T and whose proof fails rarely enough: the proof fails when
// some block has an element of the row's top k in every group; with x_k = k * (1024 / G) / V elements
// of the top k per group that happens with probability about Nb * (1 - exp(-x_k))^m per row, which must
// stay below 1e-3 (warp mode with four groups would send one row in three hundred to the exact kernel at
// k = 64, V = 2^18, and such a row costs more than the whole call does without it).  Tile mode stops at
// G = 8: a minimum over more groups now and then falls so low that the tile overflows its candidate slot.
// Returns G, plus PICK_TILE_MODE in tile mode; 0 means "keep every finite element" (vocabularies the
// merge can sort whole); -1 hands the row to the exact kernel.
#ifndef SONIC_LG_FAIL_MAX
#define SONIC_LG_FAIL_MAX -9.97f          // log2(1e-3)
#endif
constexpr int PICK_TILE_MODE = 0x100;
__device__ __forceinline__ int pick_groups(int k, int V) {
    if (V <= MERGE_CAP) return 0;
    const float lg_nw = __log2f((float)((V + WARP_TILE - 1) / WARP_TILE));
    const float lg_nt = __log2f((float)((V + CTA_TILE - 1) / CTA_TILE));
    for (int step = 0; step < 11; ++step) {
        const bool tile = (step & 1) != 0;
        if (tile && step > 7) continue;
        const int G = tile ? (1 << (step >> 1)) : (2 << (step >> 1));
        const float m = (float)(tile ? G * (CTA_TILE / WARP_TILE) : G);              // groups per block
        const float lg = tile ? lg_nt : lg_nw;                                      // log2 of the blocks per row
        const float r = exp2f(-lg / m);                                             // Nb^(-1/m)
        const float est = (float)V * ((float)G / (float)WARP_TILE) * -__logf(1.0f - r);
        // the proven count scatters around the estimate (about 15 % at 16 groups, far more at 2)
        const float need = (float)k * (m >= 16.0f ? 1.7f : 1.0f + 6.0f * rsqrtf(m)) + 30.0f;
        // above MERGE_CAP the merge first narrows the candidates with a key floor; the tiles' slots bound the rest
        const float xk = (float)k * ((float)WARP_TILE / (float)G) / (float)V;
        const float lg_fail = lg + m * __log2f(1.0f - __expf(-xk));                 // log2 of the failure probability
        if (est >= need && lg_fail <= SONIC_LG_FAIL_MAX)
            return (est <= 0.5f * (float)CAND_CAP) ? (G | (tile ? PICK_TILE_MODE : 0)) : -1;
    }
    return -1;
}

// The per-request parameters as read from global memory.  Every array that exists is read at once (one
// global-memory latency, not a chain behind the mode word); values whose mode bit is clear are dropped by
// resolve_cfg.
struct CfgRaw {
    uint32_t z;
    float tau, p, theta, alpha, beta, gamma;
    int k, hl, bl;
};
__device__ __forceinline__ CfgRaw fetch_cfg(const KParams &P, int row) {
    const int b = (P.op == OP_VERIFY) ? row / (P.K + 1) : row;
    CfgRaw r;
    r.z = (P.op == OP_TOPK) ? M_TOP_K : P.mode[b];
    r.tau = P.temperature ? P.temperature[b] : 1.0f;
    r.k = (P.op != OP_TOPK && P.top_k) ? P.top_k[b] : 0;
    r.p = P.top_p ? P.top_p[b] : 1.0f;
    r.theta = P.min_p ? P.min_p[b] : 0.0f;
    r.alpha = P.rep ? P.rep[b] : 1.0f;
    r.beta = P.freq ? P.freq[b] : 0.0f;
    r.gamma = P.pres ? P.pres[b] : 0.0f;
    r.hl = P.hist_len ? P.hist_len[b] : 0;
    r.bl = P.bias_len ? P.bias_len[b] : 0;
    return r;
}

// memo_k / memo_G: the caller's memory of the last (k, G) pair, so that runs of rows with one k skip pick_groups
__device__ __forceinline__ RowCfg resolve_cfg(const KParams &P, int row, const CfgRaw &raw, int *memo_k = nullptr, int *memo_G = nullptr) {
    RowCfg c;
    c.b = row; c.l = 0;
    if (P.op == OP_VERIFY) { c.b = row / (P.K + 1); c.l = row - c.b * (P.K + 1); }
    const uint32_t z_in = raw.z;
    const float v_tau = raw.tau, v_p = raw.p, v_theta = raw.theta, v_alpha = raw.alpha, v_beta = raw.beta, v_gamma = raw.gamma;
    const int v_k = raw.k, v_hl = raw.hl, v_bl = raw.bl;
    c.z = z_in;
    uint32_t z = c.z;
    c.bad = false;
    // a set bit whose parameter array is missing cannot be honoured
    if ((z & M_TEMPERATURE) && !P.temperature) { c.bad = true; z &= ~M_TEMPERATURE; }
    if (P.op != OP_TOPK && (z & M_TOP_K) && !P.top_k) { c.bad = true; z &= ~M_TOP_K; }
    if ((z & M_TOP_P) && !P.top_p) { c.bad = true; z &= ~M_TOP_P; }
    if ((z & M_MIN_P) && !P.min_p) { c.bad = true; z &= ~M_MIN_P; }
    if ((z & M_REPETITION) && !P.rep) { c.bad = true; z &= ~M_REPETITION; }
    if ((z & M_FREQUENCY) && !P.freq) { c.bad = true; z &= ~M_FREQUENCY; }
    if ((z & M_PRESENCE) && !P.pres) { c.bad = true; z &= ~M_PRESENCE; }
    if ((z & M_PENALTIES) && !(P.hist_ids && P.hist_counts && P.hist_len)) { c.bad = true; z &= ~M_PENALTIES; }
    if ((z & M_BIAS) && !(P.bias_ids && P.bias_vals && P.bias_len)) { c.bad = true; z &= ~M_BIAS; }
    if ((z & M_GRAMMAR) && !P.bitmask) { c.bad = true; z &= ~M_GRAMMAR; }
    c.z = z;
    c.temp = (z & M_TEMPERATURE) != 0;
    c.tau = c.temp ? v_tau : 1.0f;
    c.k = (P.op == OP_TOPK) ? P.ktop : ((z & M_TOP_K) ? v_k : 0);
    c.p = (z & M_TOP_P) ? v_p : 1.0f;
    c.theta = (z & M_MIN_P) ? v_theta : 0.0f;
    c.alpha = (z & M_REPETITION) ? v_alpha : 1.0f;
    c.beta = (z & M_FREQUENCY) ? v_beta : 0.0f;
    c.gamma = (z & M_PRESENCE) ? v_gamma : 0.0f;
    c.hist_len = (z & M_PENALTIES) ? min(max(v_hl, 0), P.hist_stride) : 0;   // never past the request's slice
    c.bias_len = (z & M_BIAS) ? min(max(v_bl, 0), P.bias_stride) : 0;
    bool greedy = (z & M_GREEDY) != 0;
    if (c.temp && !(c.tau > 0.0f && c.tau < CUDART_INF_F)) c.bad = true;
    // penalty coefficients (Appendix "Repetition Penalties" states alpha >= 1 and beta, gamma >= 0): a divisor that is not
    // positive and finite, or a coefficient that is not finite, would turn logits into NaN or +-inf
    if ((z & M_REPETITION) && !(c.alpha > 0.0f && c.alpha < CUDART_INF_F)) c.bad = true;
    if ((z & M_FREQUENCY) && !(fabsf(c.beta) < CUDART_INF_F)) c.bad = true;
    if ((z & M_PRESENCE) && !(fabsf(c.gamma) < CUDART_INF_F)) c.bad = true;
    if (!greedy) {
        if ((z & M_TOP_K) && c.k < 0) c.bad = true;
        if ((z & M_TOP_P) && !(c.p > 0.0f && c.p <= 1.0f)) c.bad = true;
        if ((z & M_MIN_P) && !(c.theta > 0.0f && c.theta <= 1.0f)) c.bad = true;
    }
    if (c.k < 0) c.k = 0;
    // TopP with p = 1 keeps every survivor of the other filters (the whole mass is reached by the whole set only; in
    // floating point the comparison would be decided by rounding): the bit is dropped
    if ((z & M_TOP_P) && c.p >= 1.0f) { z &= ~M_TOP_P; c.z = z; c.p = 1.0f; }
    c.div_all = false;
    c.G = 0;
    c.tile_min = false;
    if (greedy || (P.op == OP_TOPK && c.k == 1)) {
        c.cls = CLS_GREEDY;
        c.div_all = c.temp;
    } else {
        int kfast = (P.op == OP_TOPK) ? KFAST_TOPK : KFAST_SAMPLE;
        c.cls = CLS_EXACT;
        if (c.k == 0 && P.op != OP_TOPK) {
            c.cls = CLS_DENSE;                 // the keys it stores are final: divided by the temperature
            c.div_all = c.temp;
        } else if (c.k > 0 && c.k <= kfast) {
            int G;
            if (memo_k && *memo_k == c.k) G = *memo_G;
            else {
                G = pick_groups(c.k, P.V);
                if (memo_k) { *memo_k = c.k; *memo_G = G; }
            }
            if (G >= 0) { c.cls = CLS_TOPK; c.G = G & (PICK_TILE_MODE - 1); c.tile_min = (G & PICK_TILE_MODE) != 0; }
        }
    }
    return c;
}

__device__ __forceinline__ RowCfg load_cfg(const KParams &P, int row) { return resolve_cfg(P, row, fetch_cfg(P, row)); }

#ifdef SONIC_TRACE
__device__ __forceinline__ unsigned int gtimer_lo() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return (unsigned int)t; }
// kernel-level timeline (trace variant of the library only): earliest start and latest end of kernel k over its CTAs
// (0 stream, 1 merge, 6 histogram pass, 3 collect pass, 8 row finish, 4 residual pass, 9 residual draw, 2 cluster kernel, 5 combine)
#define KERNEL_T0(k) do { if (threadIdx.x == 0) atomicMin(&P.error[48 + 2 * (k)], gtimer_lo()); } while (0)
#define KERNEL_T1(k) do { if (threadIdx.x == 0) atomicMax(&P.error[49 + 2 * (k)], gtimer_lo()); } while (0)
#else
#define KERNEL_T0(k) do { } while (0)
#define KERNEL_T1(k) do { } while (0)
#endif

// ---------------------------------------------------------------- Philox4x32-10
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 24-bit cell index of the two uniforms of (seed, position, request):
// u = (a + 1/2) / 2^24, word 0 for the accept test, word 1 for the draw.
__device__ __forceinline__ void draw_cells(const KParams &P, const RowCfg &c, uint32_t &a_accept, uint32_t &a_draw) {
    unsigned long long seed = P.seed ? P.seed[c.b] : 0ull;
    unsigned long long pos = (P.offset ? P.offset[c.b] : 0ull) + (unsigned long long)c.l;
    uint32_t r[4];
    philox4x32_10((uint32_t)pos, (uint32_t)(pos >> 32), (uint32_t)c.b, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), r);
    a_accept = r[0] >> 8;
    a_draw = r[1] >> 8;
}
__device__ __forceinline__ double cell_to_u(uint32_t a) { return ((double)a + 0.5) * (1.0 / 16777216.0); }

// Penalties of one history token, in the paper's order, one rounding per operator.
__device__ __forceinline__ float apply_penalties(float v, int count, const RowCfg &c) {
    if (count <= 0) return v;
    if (c.z & M_REPETITION) v = (v > 0.0f) ? __fdiv_rn(v, c.alpha) : __fmul_rn(v, c.alpha);
    if (c.z & M_FREQUENCY) v = __fsub_rn(v, __fmul_rn(c.beta, (float)count));
    if (c.z & M_PRESENCE) v = __fsub_rn(v, c.gamma);
    return v;
}

__device__ __forceinline__ unsigned long long ldcg_u64(const unsigned long long *p) {
    return __ldcg(p);
}

// Writes the per-row outputs of the sample / verify operations.
__device__ __forceinline__ void emit_row(const KParams &P, const RowCfg &c, int row, int token, float prob,
                                         uint32_t flags, int support, float p_draft) {
    if (P.op == OP_SAMPLE) {
        P.out_token[row] = token;
        P.out_prob[row] = prob;
        P.out_flags[row] = flags;
        if (P.out_support) P.out_support[row] = support;
    } else {
        PosResult r;
        r.token = token; r.flags = flags; r.p = p_draft; r.support = support;
        P.pr[row] = r;
    }
}

// Fixed-point softmax weight of a key relative to the row maximum: 2^40 * exp(y - M).  Sums of these are
// order-independent, so replays are bit-identical.  Callers weigh every element and select afterwards
// (w = qweight(key); sum += cond ? w : 0): behind a branch per element the sixteen independent chains of a thread
// cannot overlap and a pass takes four times as long.
__device__ __forceinline__ unsigned long long qweight(uint32_t key, float Mf) {
    float d = __fsub_rn(unkey(key), Mf);
    const float L1 = 1.44269502162933349609375f;        // fp32(log2 e)
    const float L2 = 1.925963033500011e-08f;            // log2 e - L1
    float t = fmaf(d, L1, d * L2);
    float w;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(w) : "f"(t));
    return __float2ull_rn(w * 1099511627776.0f);
}

// exp(d) for d <= 0 in fp32 with a relative error below 1e-7 and no bias to speak of (mean 4e-10): d * log2(e) is
// split into its nearest integer and a fraction in [-1/2, 1/2] by one fused multiply-add (so the error does not grow
// with |d|), 2^fraction is a degree-6 polynomial, the integer goes into the exponent field.  Used where fp64 is too
// slow to weigh every element (the residual pass) and ex2.approx is too coarse.
__device__ __forceinline__ float exp_accurate(float d) {
    d = fmaxf(d, -80.0f);
    const float L1 = 1.44269502162933349609375f;        // fp32(log2 e)
    const float L2 = 1.925963033500011e-08f;            // log2 e - L1
    const float MAGIC = 12582912.0f;                     // 1.5 * 2^23: adding it leaves the nearest integer in the low mantissa bits
    const float r = fmaf(d, L1, MAGIC);
    const int ei = __float_as_int(r) - 0x4B400000;       // round(d * log2 e), >= -116
    const float f = fmaf(d, L2, fmaf(d, L1, -__fsub_rn(r, MAGIC)));
    float p = 0.00015337577497120947f;
    p = fmaf(p, f, 0.0013399859890341759f);
    p = fmaf(p, f, 0.009618519805371761f);
    p = fmaf(p, f, 0.05550329014658928f);
    p = fmaf(p, f, 0.24022646248340607f);
    p = fmaf(p, f, 0.6931471824645996f);
    p = fmaf(p, f, 1.0f);                                // 2^f in [0.7071, 1.4143]
    return __int_as_float(__float_as_int(p) + (ei << 23));
}

// floor(W * u) for the draw's uniform u = (2 a + 1) / 2^25, exactly.
__device__ __forceinline__ unsigned long long draw_target(unsigned long long W, uint32_t a_draw) {
    const unsigned long long mul = 2ull * a_draw + 1ull;
    return (__umul64hi(W, mul) << 39) | ((W * mul) >> 25);
}

// Smallest float not below M + ln(theta) taken in double, as an ordered key: y passes min-p  <=>  okey(y) >= it.
__device__ __forceinline__ uint32_t minp_key(float Mf, float theta) {
    const double thr = (double)Mf + log((double)theta);
    float tf = (float)thr;
    if ((double)tf < thr) tf = nextafterf(tf, CUDART_INF_F);
    return okey(tf);
}

// Programmatic dependent launch (the paper overlaps its two stages the same way, Section 3.5):
// a kernel lets the next kernel of the stream start launching early, and that kernel waits
// here until the previous one has completed and its writes are visible.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_primary() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Block-level barriers: the whole CTA, or only the 256 consumer threads of the
// streaming kernel (named barrier 1; its producer warp never joins).
struct BlockSync { __device__ __forceinline__ void operator()() const { __syncthreads(); } };
struct ConsumerSync {
    __device__ __forceinline__ void operator()() const { asm volatile("bar.sync 1, 256;" ::: "memory"); }
};

// Descending bitonic sort of m (power of two) 64-bit keys in shared memory.
// The 32 lanes of a warp always work on one aligned block of 64 keys when the
// partner distance j is at most 32, so those stages only need a warp barrier;
// the block barrier is kept around the stages with j >= 64.
template <int THREADS, typename Sync = BlockSync>
__device__ __forceinline__ void bitonic_sort_desc(unsigned long long *a, int m, int tid) {
    Sync sync;
    for (int k2 = 2; k2 <= m; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < (m >> 1); i += THREADS) {
                int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
                int hi = lo | j;
                unsigned long long x = a[lo], y = a[hi];
                bool desc = ((lo & k2) == 0);
                if ((x < y) == desc) { a[lo] = y; a[hi] = x; }
            }
            const int jn = (j > 1) ? (j >> 1) : k2;          // partner distance of the next stage
            if (j >= 64 || jn >= 64 || (k2 == m && j == 1)) sync(); else __syncwarp();
        }
    }
}

// The same sort by a whole CTA, with every thread holding two adjacent elements in registers: the stages whose
// partner distance is at most 32 run on shuffles (distance 1 inside the thread) and only the wider ones go
// through shared memory with a block barrier.  m is a power of two; zeros may pad the tail.  Not inlined and
// with rolled loops: one compact copy of the code serves every caller.
template <int THREADS>
__device__ __noinline__ void bitonic_sort_desc_cta(unsigned long long *a, int m, int tid) {
    const int mm = max(m, 64);                           // whole warps take part (64 elements each)
    auto tail = [&](unsigned long long &x0, unsigned long long &x1, int e, int k2, int jtop) {
        const bool desc = ((e & k2) == 0);
#pragma unroll 1
        for (int j = jtop; j >= 2; j >>= 1) {
            const unsigned long long o0 = __shfl_xor_sync(0xFFFFFFFFu, x0, j >> 1);
            const unsigned long long o1 = __shfl_xor_sync(0xFFFFFFFFu, x1, j >> 1);
            const bool take_max = (desc == ((e & j) == 0));
            // keep mine if it is on the side this lane takes, else the partner's (one comparison per element)
            x0 = ((x0 > o0) == take_max) ? x0 : o0;
            x1 = ((x1 > o1) == take_max) ? x1 : o1;
        }
        if ((x0 > x1) != desc) { const unsigned long long t = x0; x0 = x1; x1 = t; }
    };
#pragma unroll 1
    for (int base = 0; base < mm; base += 2 * THREADS) {
        const int e = base + 2 * tid;
        if (e < mm) {                                    // uniform over the warp
            unsigned long long x0 = (e < m) ? a[e] : 0ull, x1 = (e + 1 < m) ? a[e + 1] : 0ull;
#pragma unroll 1
            for (int k2 = 2; k2 <= 64; k2 <<= 1) tail(x0, x1, e, k2, k2 >> 1);
            if (e < m) a[e] = x0;
            if (e + 1 < m) a[e + 1] = x1;
        }
    }
    __syncthreads();
#pragma unroll 1
    for (int k2 = 128; k2 <= mm; k2 <<= 1) {
#pragma unroll 1
        for (int j = k2 >> 1; j >= 64; j >>= 1) {
            for (int i = tid; i < (mm >> 1); i += THREADS) {
                const int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
                const int hi = lo | j;
                const unsigned long long x = a[lo], y = a[hi];
                const bool desc = ((lo & k2) == 0);
                if ((x < y) == desc) { a[lo] = y; a[hi] = x; }
            }
            __syncthreads();
        }
#pragma unroll 1
        for (int base = 0; base < mm; base += 2 * THREADS) {
            const int e = base + 2 * tid;
            if (e < mm) {
                unsigned long long x0 = a[e], x1 = a[e + 1];
                tail(x0, x1, e, k2, 32);
                a[e] = x0; a[e + 1] = x1;
            }
        }
        __syncthreads();
    }
}

// Ranks of at most THREADS distinct non-zero keys held one per thread in list[0, n): every warp sorts its 32 keys
// with shuffles and writes them back as a descending run, then a key's rank is its place in its own run plus, for
// every other run, the number of keys there above it (a binary search in the sorted run; 0 pads the last run).
// Returns the thread's key after the warp sort (0 = padding) and leaves its rank in `rank`.  Two block barriers.
template <int THREADS, typename Sync>
__device__ __forceinline__ unsigned long long rank_keys(unsigned long long *list, int n, int tid, int &rank) {
    Sync csync;
    const int lane = tid & 31, warp = tid >> 5;
    unsigned long long key = (tid < n) ? list[tid] : 0ull;
#pragma unroll
    for (int kk = 2; kk <= 32; kk <<= 1) {
#pragma unroll
        for (int jj = kk >> 1; jj > 0; jj >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, key, jj);
            const bool up = ((lane & kk) == 0);            // this block of kk sorts descending
            const bool first = ((lane & jj) == 0);         // the lower lane of the pair
            const bool take_max = (up == first);
            key = ((key > o) == take_max) ? key : o;           // mine if it is on the side this lane takes
        }
    }
    csync();                                               // every thread has read its key from the list
    list[tid] = key;                                       // sorted runs of 32 (descending), in place
    csync();
    const int runs = (n + 31) >> 5;
    rank = lane;
    if (key != 0ull) {
        // four runs at a time: their binary searches are independent chains of shared-memory reads
        for (int r0 = 0; r0 < runs; r0 += 4) {
            const unsigned long long *run[4];
            int lo[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { run[u] = list + min(r0 + u, runs - 1) * 32; lo[u] = 0; }
#pragma unroll
            for (int step = 16; step > 0; step >>= 1) {
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (run[u][lo[u] + step - 1] > key) lo[u] += step;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (lo[u] < 32 && run[u][lo[u]] > key) ++lo[u];        // covers a run whose 32 keys are all above
                if (r0 + u < runs && r0 + u != warp) rank += lo[u];     // (lo[u] = number of keys of the run above `key`)
            }
        }
    }
    return key;
}

__device__ __forceinline__ int next_pow2(int n) {
    int m = 2;
    while (m < n) m <<= 1;
    return m;
}

// Inclusive scan of n doubles in shared memory (in place), THREADS threads,
// fixed evaluation order (deterministic).  `scratch` holds THREADS doubles.
template <int THREADS, typename Sync = BlockSync>
__device__ __forceinline__ void block_inclusive_scan(double *v, int n, double *scratch, int tid) {
    Sync sync;
    int chunk = (n + THREADS - 1) / THREADS;
    int lo = tid * chunk, hi = min(lo + chunk, n);
    double s = 0.0;
    for (int i = lo; i < hi; ++i) { s += v[i]; v[i] = s; }
    scratch[tid] = s;
    sync();
    if (tid < 32) {
        // serial over 32 segments of THREADS/32 partials each: short and order-fixed
        constexpr int PER = THREADS / 32;
        double loc = 0.0;
        for (int i = 0; i < PER; ++i) { double t = scratch[tid * PER + i]; scratch[tid * PER + i] = loc; loc += t; }
        double incl = loc;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            double o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (tid >= off) incl += o;
        }
        double excl = incl - loc;
        for (int i = 0; i < PER; ++i) scratch[tid * PER + i] += excl;
    }
    sync();
    double off = scratch[tid];
    for (int i = lo; i < hi; ++i) v[i] += off;
    sync();
}

}  // namespace sonic
