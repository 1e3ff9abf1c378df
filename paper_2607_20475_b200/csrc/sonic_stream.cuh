// Streaming kernel: reads every logit of the rows it owns exactly once, applies
// the logit-processing prologue, and reduces each 8192-element tile either to
// an argmax (greedy rows) or to the complete set of elements above a tile
// cutoff (top-k rows), written to the tile's own slot of the workspace without
// atomics.  The CTA that finishes a row's last tile merges the row (global
// top-k, truncation epilogue, token selection) while the others keep streaming.
// The two halves correspond to the paper's Algorithms "Stage 1: Tile-Local
// Reduction Kernel" and "Stage 2: Cross-Tile Merge and Selection Kernel"; the
// selection itself is ours.
//
// Structure: persistent CTAs (two per SM), each a producer warp plus eight
// consumer warps.  The producer walks the CTA's tiles, resolves each tile's row
// configuration and issues one bulk-TMA copy (cp.async.bulk, completion on an
// mbarrier) of the tile's logits into a ring of shared-memory stages, several
// tiles ahead of the consumers, so HBM requests stay in flight while the
// consumers compute.  Every mbarrier wait is bounded: on expiry the kernel
// records an error in the workspace header and returns.
//
// Exactness: a tile's cutoff t is the minimum of G group maxima, so at least G
// of its elements are >= t, and the tile emits EVERY finite element >= t.  With
// T the largest cutoff of the row, the emitted elements >= T are exactly the
// row's elements >= T.  If there are at least k of them the row's top-k is
// their top-k; otherwise the row is handed to the exact kernel.
#pragma once
#include "sonic_common.cuh"

namespace sonic {

template <int DT> struct VecTraits;
template <> struct VecTraits<0> { static constexpr int VEC = 4, NV = 8, NSTAGE = 2, ELT = 4; };
template <> struct VecTraits<1> { static constexpr int VEC = 8, NV = 4, NSTAGE = 2, ELT = 2; };

constexpr int STREAM_CTA_THREADS = STREAM_THREADS + 32;      // eight consumer warps + the producer warp
constexpr unsigned int WAIT_LIMIT = 1u << 22;                // try_wait rounds before a wait gives up

// ---------------------------------------------------------------- mbarrier / bulk-copy primitives
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *bar, unsigned int bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false if it did not complete in time.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned int parity) {
    const uint32_t addr = smem_u32(bar);
    for (unsigned int it = 0; it < WAIT_LIMIT; ++it) {
        unsigned int done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
// One bulk copy global -> this CTA's shared memory; bytes and both addresses are multiples of 16.
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned int bytes, unsigned long long *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Element index of register slot s of a lane.
template <int DT>
__device__ __forceinline__ int slot_index(int wbase, int lane, int s) {
    constexpr int VEC = VecTraits<DT>::VEC;
    return wbase + (s / VEC) * 32 * VEC + lane * VEC + (s % VEC);
}

template <int THREADS>
struct MergeShared {
    int count;
    int tcnt[MAX_TILES + 1];                   // exclusive prefix of the tiles' candidate counts
    unsigned int tkey;
    int n_p, n_m, pick;
    int found;
    double scratch[THREADS];
};

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

#ifdef SONIC_TRACE
#define MERGE_STAMP(i) do { if (tid == 0 && row == (int)P.error[4]) P.error[8 + (i)] = (unsigned int)clock64(); } while (0)
#else
#define MERGE_STAMP(i) do { } while (0)
#endif

constexpr int RANK_SORT_MAX = 512;            // at most this many candidates: sort by rank counting
constexpr int WARP_EPILOGUE_MAX = 128;        // at most this many survivors of TopK: one warp finishes the row
struct WarpSync { __device__ __forceinline__ void operator()() const { __syncwarp(); } };

template <int NT, typename Sync, typename SH>
__device__ void merge_epilogue(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid);

// Row merge for top-k class rows (one CTA per row).  buf is MERGE_CAP 64-bit
// words of shared memory.  Returns false if the candidates cannot prove the
// row's answer.
template <int THREADS, typename Sync>
__device__ bool merge_topk_row(const KParams &P, const RowCfg &c, int row, int tiles,
                               unsigned long long *buf, MergeShared<THREADS> &sh, int tid) {
    Sync csync;
    MERGE_STAMP(0);
    const int cap_t = (int)(CAND_CAP / (unsigned)tiles);
    const TileRec *rec = P.tiles + (size_t)row * MAX_TILES;
    // tile records: one thread per tile, then a serial prefix over at most 32 entries
    if (tid == 0) { sh.count = 0; sh.tkey = 0; sh.found = 0; }
    csync();
    if (tid < tiles) {
        const unsigned int cnt = __ldcg(&rec[tid].cnt);
        P.tiles[(size_t)row * MAX_TILES + tid].cnt = 0u;           // the streaming kernel accumulates into it
        sh.tcnt[tid + 1] = (int)cnt;
        atomicMax(&sh.tkey, __ldcg(&rec[tid].tkey));
        if (cnt > (unsigned int)cap_t) sh.found = 1;     // a tile overflowed its slot
    }
    csync();
    if (sh.found) return false;
    if (tid == 0) {
        sh.tcnt[0] = 0;
        for (int t = 0; t < tiles; ++t) sh.tcnt[t + 1] += sh.tcnt[t];
    }
    csync();
    MERGE_STAMP(1);
    const unsigned int tkey = sh.tkey;
    const bool complete = (tkey == KEY_NEG_INF);
    const bool strict = c.temp && !complete;            // keys are compared after the temperature division
    const uint32_t tykey = c.temp ? okey(__fdiv_rn(unkey(tkey), c.tau)) : tkey;
    const int total = sh.tcnt[tiles];
    // candidates are fetched eight per thread at a time (independent loads), then filtered and packed
    constexpr int GB = 8;
    auto fetch = [&](int j0, unsigned long long (&cd)[GB]) {
#pragma unroll
        for (int u = 0; u < GB; ++u) {
            const int j = j0 + u * THREADS + tid;
            cd[u] = 0ull;
            if (j < total) {
                int t = 0;
                while (sh.tcnt[t + 1] <= j) ++t;
                cd[u] = __ldcg(P.cand + (size_t)row * CAND_CAP + (size_t)t * cap_t + (j - sh.tcnt[t]));
            }
        }
    };
    // proven candidate -> its key after the temperature division (0 if it is not proven)
    auto proven_key = [&](unsigned long long cd, int j) -> unsigned long long {
        const uint32_t zk = (uint32_t)(cd >> 32);
        uint32_t yk = zk;
        if (c.temp) yk = okey(__fdiv_rn(unkey(zk), c.tau));
        const bool keep = (j < total) && (zk >= tkey) && !(strict && yk <= tykey);
        return keep ? (((unsigned long long)yk << 32) | (uint32_t)cd) : 0ull;
    };
    unsigned long long floor_key = 1ull;           // keys below it are left out (1: every proven candidate)
    for (int attempt = 0; attempt < 2; ++attempt) {
        unsigned long long kmax = 0ull;
        for (int j0 = 0; j0 < total; j0 += GB * THREADS) {
            unsigned long long cd[GB];
            fetch(j0, cd);
#pragma unroll
            for (int u = 0; u < GB; ++u) {
                if (j0 + u * THREADS >= total) break;              // uniform over the CTA
                const unsigned long long out = proven_key(cd[u], j0 + u * THREADS + tid);
                const bool keep = out >= floor_key;
                kmax = max(kmax, out);
                // one shared-memory atomic per warp, not per candidate
                const unsigned int m = __ballot_sync(0xFFFFFFFFu, keep);
                int base = 0;
                if ((tid & 31) == 0 && m) base = atomicAdd(&sh.count, __popc(m));
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
                if (keep) {
                    const int pos = base + __popc(m & ((1u << (tid & 31)) - 1u));
                    if (pos < MERGE_CAP) buf[pos] = out;
                }
            }
        }
        csync();
        if (attempt == 1 || sh.count <= MERGE_CAP || sh.count < c.k) break;
        // More proven candidates than the buffer holds (large k): find a key floor that keeps between k and
        // MERGE_CAP of them by an eight-way search over the candidates in global memory, then pack again.
        unsigned long long *red = reinterpret_cast<unsigned long long *>(sh.scratch);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, off));
        if ((tid & 31) == 0) red[tid >> 5] = kmax;
        csync();
        for (int w = 0; w < THREADS / 32; ++w) kmax = max(kmax, red[w]);
        csync();
        unsigned long long lo = 1ull, hi = kmax + 1ull;              // count(>= lo) >= k > ... count(>= hi) = 0
        for (int it = 0; it < 24 && hi - lo > 1ull; ++it) {
            const unsigned long long step = (hi - lo) >> 3;
            unsigned long long th[7];
#pragma unroll
            for (int q = 0; q < 7; ++q) th[q] = (step > 0) ? lo + step * (q + 1) : min(hi - 1ull, lo + 1ull + q);
            int cnt[7] = {0, 0, 0, 0, 0, 0, 0};
            for (int j0 = 0; j0 < total; j0 += GB * THREADS) {
                unsigned long long cd[GB];
                fetch(j0, cd);
#pragma unroll
                for (int u = 0; u < GB; ++u) {
                    const unsigned long long out = proven_key(cd[u], j0 + u * THREADS + tid);
#pragma unroll
                    for (int q = 0; q < 7; ++q) cnt[q] += (out >= th[q]) ? 1 : 0;
                }
            }
            int *redi = reinterpret_cast<int *>(sh.scratch);
#pragma unroll
            for (int q = 0; q < 7; ++q) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) cnt[q] += __shfl_xor_sync(0xFFFFFFFFu, cnt[q], off);
                if ((tid & 31) == 0) redi[(tid >> 5) * 8 + q] = cnt[q];
            }
            csync();
            bool done = false;
            bool fits = false;
#pragma unroll
            for (int q = 6; q >= 0; --q) {                 // the highest threshold that still keeps k
                int tot = 0;
                for (int w = 0; w < THREADS / 32; ++w) tot += redi[w * 8 + q];
                if (!done && tot >= c.k) {
                    lo = th[q];
                    if (q < 6) hi = th[q + 1];
                    done = true;
                    fits = tot <= MERGE_CAP;
                }
            }
            if (!done) hi = th[0];
            csync();
            if (fits) break;
        }
        floor_key = lo;
        if (tid == 0) sh.count = 0;
        csync();
    }
    csync();
    const int Pn = sh.count;
    MERGE_STAMP(2);
    if (Pn > MERGE_CAP) return false;
    int n;
    if (Pn >= c.k) n = c.k;
    else if (complete && P.op != OP_TOPK) n = Pn;
    else return false;
    unsigned long long *sorted = buf;
    int Pn2 = Pn;
    if (Pn > RANK_SORT_MAX && Pn > n + n / 2 + 64) {
        // far more proven candidates than needed: bisect a key threshold that keeps between n and
        // about next_pow2(n) of them (any such threshold keeps the n best), then sort only those
        const int want_hi = next_pow2(n);                   // so that the sort below runs on the smallest power of two
        unsigned long long lo = 0ull, hi = ~0ull;          // count(>= lo) >= n > count(>= hi)
        {
            // start from the range the keys actually span
            unsigned long long mn = ~0ull, mx = 0ull;
            for (int i = tid; i < Pn; i += THREADS) { mn = min(mn, buf[i]); mx = max(mx, buf[i]); }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                mn = min(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
                mx = max(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
            }
            unsigned long long *red = reinterpret_cast<unsigned long long *>(sh.scratch);
            if ((tid & 31) == 0) { red[tid >> 5] = mn; red[THREADS / 32 + (tid >> 5)] = mx; }
            csync();
            for (int w = 0; w < THREADS / 32; ++w) { mn = min(mn, red[w]); mx = max(mx, red[THREADS / 32 + w]); }
            csync();
            lo = mn; hi = mx + 1ull;
        }
        MERGE_STAMP(11);
        // eight-way search: seven interior thresholds per pass, one reduction for all of them
        for (int it = 0; it < 24 && hi - lo > 1ull; ++it) {
            const unsigned long long step = (hi - lo) >> 3;
            unsigned long long th[7];
#pragma unroll
            for (int q = 0; q < 7; ++q) th[q] = (step > 0) ? lo + step * (q + 1) : min(hi - 1ull, lo + 1ull + q);
            int cnt[7] = {0, 0, 0, 0, 0, 0, 0};
            for (int i = tid; i < Pn; i += THREADS) {
                const unsigned long long key = buf[i];
#pragma unroll
                for (int q = 0; q < 7; ++q) cnt[q] += (key >= th[q]) ? 1 : 0;
            }
            int *redi = reinterpret_cast<int *>(sh.scratch);
#pragma unroll
            for (int q = 0; q < 7; ++q) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) cnt[q] += __shfl_xor_sync(0xFFFFFFFFu, cnt[q], off);
                if ((tid & 31) == 0) redi[(tid >> 5) * 8 + q] = cnt[q];
            }
            csync();
            bool done = false;
#pragma unroll
            for (int q = 6; q >= 0; --q) {                 // the highest threshold that still keeps n
                int tot = 0;
                for (int w = 0; w < THREADS / 32; ++w) tot += redi[w * 8 + q];
                if (!done && tot >= n) {
                    lo = th[q];
                    if (q < 6) hi = th[q + 1];
                    done = true;
                    if (tot <= want_hi) it = 1000;          // tight enough
                }
            }
            if (!done) hi = th[0];
            csync();
        }
        // keep the keys >= lo, packed to the front (every position written is at or below one already read)
        if (tid == 0) sh.count = 0;
        csync();
        for (int i0 = 0; i0 < Pn; i0 += THREADS) {
            const int i = i0 + tid;
            const unsigned long long key = (i < Pn) ? buf[i] : 0ull;
            const bool keep = (i < Pn) && key >= lo;
            const unsigned int mk = __ballot_sync(0xFFFFFFFFu, keep);
            csync();                                        // all reads of this trip precede its writes
            int base = 0;
            if ((tid & 31) == 0 && mk) base = atomicAdd(&sh.count, __popc(mk));
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if (keep) buf[base + __popc(mk & ((1u << (tid & 31)) - 1u))] = key;
            csync();
        }
        Pn2 = sh.count;
        csync();
    }
    MERGE_STAMP(12);
#ifdef SONIC_TRACE
    if (tid == 0 && row == (int)P.error[4]) P.error[29] = Pn2;
#endif
    const int PnAll = Pn;
    (void)PnAll;
#define Pn Pn2
    if (Pn <= RANK_SORT_MAX) {
        // few candidates: each key counts the keys above it (keys are distinct) and lands at its rank
        unsigned long long *dst = buf + MERGE_CAP / 2;
        for (int i = tid; i < Pn; i += THREADS) {
            const unsigned long long key = buf[i];
            int rank = 0;
            int j = 0;
            for (; j + 8 <= Pn; j += 8) {                  // eight independent broadcast reads per trip
                unsigned long long o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) o[u] = buf[j + u];
#pragma unroll
                for (int u = 0; u < 8; ++u) rank += (o[u] > key) ? 1 : 0;
            }
            for (; j < Pn; ++j) rank += (buf[j] > key) ? 1 : 0;
            dst[rank] = key;
        }
        csync();
        for (int i = tid; i < Pn; i += THREADS) buf[i] = dst[i];
        csync();
    } else {
        const int m = next_pow2(Pn);
        for (int i = Pn + tid; i < m; i += THREADS) buf[i] = 0ull;
        csync();
        bitonic_sort_desc<THREADS, Sync>(buf, m, tid);
    }
    (void)sorted;
#undef Pn
    MERGE_STAMP(3);
#ifdef SONIC_TRACE
    if (tid == 0 && row == (int)P.error[4]) { P.error[30] = Pn; P.error[31] = n; }
#endif

    if (P.op == OP_TOPK) {
        for (int j = tid; j < n; j += THREADS) {
            unsigned long long kv = buf[j];
            P.out_vals[(size_t)row * P.ktop + j] = unkey((uint32_t)(kv >> 32));
            P.out_idx[(size_t)row * P.ktop + j] = (int)(~(uint32_t)kv);
        }
        return true;
    }
    if (n == 0) {
        if (tid == 0) emit_row(P, c, row, -1, 0.0f, F_NO_TOKEN, 0, 0.0f);
        return true;
    }
    // small supports are finished by one warp without block barriers
    if (n <= WARP_EPILOGUE_MAX) {
        if (tid < 32) merge_epilogue<32, WarpSync>(P, c, row, n, buf, sh, tid);
    } else {
        merge_epilogue<THREADS, Sync>(P, c, row, n, buf, sh, tid);
    }
    return true;
}

// Truncation epilogue and token selection over the n best candidates, sorted in
// buf[0, n) (TopK already applied): TopP, MinP, index-order CDF, Philox draw,
// and for verification rows the accept test and the residual.  Run by NT
// threads that synchronise with Sync (a whole CTA, or one warp).
template <int NT, typename Sync, typename SH>
__device__ void merge_epilogue(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid) {
    Sync csync;
    constexpr int THREADS = NT;
    // shared-memory layout after the sort (n <= KFAST_SAMPLE = MERGE_CAP / 4):
    //   buf[0, n)     sorted keys (value key << 32 | ~index)
    //   w             weights exp(y - M) in ranking order
    //   cs            cumulative sums (ranking order), later residual / CDF in index order
    //   ik            (~index << 32 | ranking position), sorted descending = index ascending
    double *w = reinterpret_cast<double *>(buf + KFAST_SAMPLE);
    double *cs = reinterpret_cast<double *>(buf + 2 * KFAST_SAMPLE);
    unsigned long long *ik = buf + 3 * KFAST_SAMPLE;
    const double M = (double)unkey((uint32_t)(buf[0] >> 32));
    for (int j = tid; j < n; j += THREADS) {
        double y = (double)unkey((uint32_t)(buf[j] >> 32));
        double wj = exp(y - M);
        w[j] = wj; cs[j] = wj;
    }
    if (tid == 0) { sh.n_p = n; sh.n_m = n; sh.found = 0; sh.pick = -1; }
    csync();
    MERGE_STAMP(4);
    block_inclusive_scan<THREADS, Sync>(cs, n, sh.scratch, tid);
    MERGE_STAMP(5);
    const double Z = cs[n - 1];
    if (c.z & M_TOP_P) {
        const double target = (double)c.p * Z;
        for (int j = tid; j < n; j += THREADS)
            if (cs[j] >= target && (j == 0 || cs[j - 1] < target)) sh.n_p = j + 1;
    }
    if (c.z & M_MIN_P) {
        const double thr = M + log((double)c.theta);
        for (int j = tid; j < n; j += THREADS) {
            bool in = (double)unkey((uint32_t)(buf[j] >> 32)) >= thr;
            bool prev_in = (j == 0) || ((double)unkey((uint32_t)(buf[j - 1] >> 32)) >= thr);
            if (!in && prev_in) sh.n_m = j;
        }
    }
    csync();
    n = min(n, min(sh.n_p, sh.n_m));
    const double W = cs[n - 1];
    csync();
    // survivors in vocabulary-index order
    MERGE_STAMP(6);
    if (n <= RANK_SORT_MAX) {
        // few survivors: each lands at the number of survivors with a smaller index
        for (int j = tid; j < n; j += THREADS) {
            const uint32_t mine = (uint32_t)buf[j];                  // ~index: larger means smaller index
            int pos = 0;
            int t = 0;
            for (; t + 8 <= n; t += 8) {
                uint32_t o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) o[u] = (uint32_t)buf[t + u];
#pragma unroll
                for (int u = 0; u < 8; ++u) pos += (o[u] > mine) ? 1 : 0;
            }
            for (; t < n; ++t) pos += ((uint32_t)buf[t] > mine) ? 1 : 0;
            ik[pos] = ((unsigned long long)mine << 32) | (unsigned long long)j;
        }
        csync();
    } else {
        const int m2 = next_pow2(n);
        for (int j = tid; j < m2; j += THREADS)
            ik[j] = (j < n) ? ((buf[j] << 32) | (unsigned long long)j) : 0ull;
        csync();
        bitonic_sort_desc<THREADS, Sync>(ik, m2, tid);
    }
    MERGE_STAMP(7);

    uint32_t a_acc, a_draw;
    draw_cells(P, c, a_acc, a_draw);
    const double u_draw = cell_to_u(a_draw);
    uint32_t flags = 0;
    float p_draft = 0.0f;
    bool use_residual = false;
    if (P.op == OP_VERIFY && c.l < P.K) {
        const int d = P.draft_tokens[(size_t)c.b * P.K + c.l];
        const float *q = P.draft_probs + ((size_t)c.b * P.K + c.l) * (size_t)P.V;
        if (tid == 0) sh.pick = -1;
        csync();
        for (int j = tid; j < n; j += THREADS)
            if ((int)(~(uint32_t)(ik[j] >> 32)) == d) sh.pick = j;
        csync();
        double Pd = 0.0;
        if (sh.pick >= 0) Pd = w[(uint32_t)ik[sh.pick]] / W;
        double Q = (d >= 0 && d < P.V) ? (double)__ldg(q + d) : 0.0;
        bool accept = (Pd > 0.0) && (cell_to_u(a_acc) * Q <= Pd);
        p_draft = (float)Pd;
        if (accept) flags |= F_ACCEPT;
        csync();
        // residual max(0, p - q) over the support, in index order
        for (int j = tid; j < n; j += THREADS) {
            int idx = (int)(~(uint32_t)(ik[j] >> 32));
            double r = w[(uint32_t)ik[j]] / W - (double)__ldg(q + idx);
            cs[j] = r > 0.0 ? r : 0.0;
        }
        csync();
        block_inclusive_scan<THREADS, Sync>(cs, n, sh.scratch, tid);
        use_residual = cs[n - 1] > 0.0;
        csync();
    }
    if (!use_residual) {
        for (int j = tid; j < n; j += THREADS) cs[j] = w[(uint32_t)ik[j]];
        csync();
        block_inclusive_scan<THREADS, Sync>(cs, n, sh.scratch, tid);
    }
    MERGE_STAMP(8);
    const double R = cs[n - 1];
    const double target = u_draw * R;
    if (tid == 0) sh.pick = n - 1;
    csync();
    for (int j = tid; j < n; j += THREADS)
        if (cs[j] > target && (j == 0 || !(cs[j - 1] > target))) sh.pick = j;
    csync();
    if (tid == 0) {
        int j = sh.pick;
        int token = (int)(~(uint32_t)(ik[j] >> 32));
        float prob = (float)(w[(uint32_t)ik[j]] / W);
        emit_row(P, c, row, token, prob, flags, n, p_draft);
    }
    MERGE_STAMP(9);
}

// What the producer hands to the consumers with each stage.
struct StageMeta {
    RowCfg cfg;
    int row, tile;
    int skip;                                  // the row belongs to the exact kernel: nothing was loaded
};

template <int DT>
struct StreamShared {
    static constexpr int NSTAGE = VecTraits<DT>::NSTAGE;
    unsigned long long full[NSTAGE];           // producer -> consumers: tile landed (transaction bytes)
    unsigned long long empty[NSTAGE];          // consumers -> producer: stage free (one arrival per consumer warp)
    StageMeta meta[NSTAGE];
    // per-stage scratch of the consumer warps (a fast warp may already be on the next tile, in the other stage)
    float tw[NSTAGE][STREAM_WARPS];
    unsigned int ncand[NSTAGE];
    unsigned long long best[NSTAGE][STREAM_WARPS];
};

template <int DT>
__global__ void __launch_bounds__(STREAM_CTA_THREADS, 3)
sonic_stream_kernel(const KParams P, const int tiles, const int nitems) {
    constexpr int VEC = VecTraits<DT>::VEC, NV = VecTraits<DT>::NV, NSTAGE = VecTraits<DT>::NSTAGE;
    constexpr int ELT = VecTraits<DT>::ELT;
    constexpr int STAGE_BYTES = CTA_TILE * ELT;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: NSTAGE raw stages | fp32 conversion tile (bf16 only) | control
    unsigned char *stages = smem_raw;
    float *conv = reinterpret_cast<float *>(smem_raw + NSTAGE * STAGE_BYTES);      // bf16 only
    StreamShared<DT> &sh = *reinterpret_cast<StreamShared<DT> *>(smem_raw + NSTAGE * STAGE_BYTES + (DT == 1 ? CTA_TILE * 4 : 0));
    ConsumerSync csync;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], STREAM_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    pdl_launch_dependents();                   // the merge kernel may start launching; it waits for this grid to finish

    if (warp == STREAM_WARPS) {
        // ------------------------------------------------------------ producer warp
        // The row configuration of the NEXT tile is resolved while the ring is still full, so that a freed
        // stage gets its bulk copy issued at once (the configuration is a chain of dependent global loads).
        int n = 0;
        int item = blockIdx.x;
        RowCfg c_next;
        if (item < nitems) c_next = load_cfg(P, item / tiles);
        for (; item < nitems; item += gridDim.x, ++n) {
            const int s = n % NSTAGE;
            const RowCfg c = c_next;
            if (n >= NSTAGE) {
                if (!mbar_wait(&sh.empty[s], ((n / NSTAGE) - 1) & 1)) {
                    if (lane == 0) atomicOr(P.error, ERR_TIMEOUT);
                    return;
                }
            }
            const int row = item / tiles, tile = item - row * tiles;
            if (lane == 0) {
                StageMeta &m = sh.meta[s];
                m.cfg = c; m.row = row; m.tile = tile; m.skip = (c.cls == CLS_EXACT) ? 1 : 0;
                if (c.cls == CLS_EXACT) {
                    mbar_arrive(&sh.full[s]);
                } else {
                    const int first = tile * CTA_TILE;
                    const int elems = min(CTA_TILE, ((P.V - first) + VEC - 1) / VEC * VEC);
                    const unsigned int bytes = (unsigned int)elems * ELT;
                    const unsigned char *src = reinterpret_cast<const unsigned char *>(P.logits) +
                                               ((size_t)row * (size_t)P.row_stride + (size_t)first) * ELT;
                    mbar_arrive_expect_tx(&sh.full[s], bytes);
                    bulk_load(stages + (size_t)s * STAGE_BYTES, src, bytes, &sh.full[s]);
                }
            }
            __syncwarp();
            const int nxt = item + gridDim.x;
            if (nxt < nitems) c_next = load_cfg(P, nxt / tiles);
        }
        return;
    }

    // ---------------------------------------------------------------- consumer warps
    int n = 0;
    for (int item = blockIdx.x; item < nitems; item += gridDim.x, ++n) {
        const int s = n % NSTAGE;
        const int row = item / tiles, tile = item - row * tiles;
        const int tile_base = tile * CTA_TILE;
        const int wbase = tile_base + warp * WARP_TILE;
        // requests that depend only on (row, tile) go out before the wait: the warp tile's 32 grammar
        // words in one coalesced load (handed to the lanes that need them by shuffles later)
        uint32_t mword = 0xFFFFFFFFu;
        if (P.bitmask) {
            const int w = (wbase >> 5) + lane;
            mword = (w < ((P.V + 31) >> 5)) ? __ldg(P.bitmask + (size_t)row * P.bitmask_stride + w) : 0u;
        }
        // the first entries of the row's sparse lists as well (lengths are checked once the configuration is known)
        const int req = (P.op == OP_VERIFY) ? row / (P.K + 1) : row;
        int h_id0 = -1, h_ct0 = 0, h_id1 = -1, h_ct1 = 0, b_id0 = -1;
        float b_v0 = 0.0f;
        const int *hid = P.hist_ids ? P.hist_ids + (size_t)req * P.hist_stride : nullptr;
        const int *hct = P.hist_counts ? P.hist_counts + (size_t)req * P.hist_stride : nullptr;
        const int *bid = P.bias_ids ? P.bias_ids + (size_t)req * P.bias_stride : nullptr;
        const float *bvl = P.bias_vals ? P.bias_vals + (size_t)req * P.bias_stride : nullptr;
        if (hid && hct) {
            if (tid < P.hist_stride) { h_id0 = __ldg(hid + tid); h_ct0 = __ldg(hct + tid); }
            if (tid + STREAM_THREADS < P.hist_stride) { h_id1 = __ldg(hid + tid + STREAM_THREADS); h_ct1 = __ldg(hct + tid + STREAM_THREADS); }
        }
        if (bid && bvl && tid < P.bias_stride) { b_id0 = __ldg(bid + tid); b_v0 = __ldg(bvl + tid); }
        if (!mbar_wait(&sh.full[s], (n / NSTAGE) & 1)) {
            if (lane == 0) atomicOr(P.error, ERR_TIMEOUT);
            return;
        }
        const StageMeta &meta = sh.meta[s];
        if (!meta.skip) {
            const RowCfg c = meta.cfg;
            RowState *rs = P.rs + row;
            TileRec *rec = P.tiles + (size_t)row * MAX_TILES + tile;
            unsigned char *stage = stages + (size_t)s * STAGE_BYTES;
            const bool masked = (c.z & M_GRAMMAR) != 0;
            const bool tail = tile_base + CTA_TILE > P.V;
            const bool patched = (c.hist_len > 0 || c.bias_len > 0);
            float *ptile = (DT == 0) ? reinterpret_cast<float *>(stage) : conv;    // fp32 view the sparse lists patch

            float e[EPL];
            auto read_raw = [&]() {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int li = warp * WARP_TILE + j * 32 * VEC + lane * VEC;
                    const uint4 raw = *reinterpret_cast<const uint4 *>(stage + (size_t)li * ELT);
                    const uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        if (DT == 0) e[j * VEC + q] = __uint_as_float(r[q]);
                        else e[j * VEC + q] = __uint_as_float((q & 1) ? (r[q >> 1] & 0xFFFF0000u) : (r[q >> 1] << 16));
                    }
                }
            };
            auto read_f32 = [&](const float *src) {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const float *p = src + warp * WARP_TILE + j * 32 * VEC + lane * VEC;
#pragma unroll
                    for (int q = 0; q < VEC; q += 4) {
                        const float4 v = *reinterpret_cast<const float4 *>(p + q);
                        e[j * VEC + q] = v.x; e[j * VEC + q + 1] = v.y; e[j * VEC + q + 2] = v.z; e[j * VEC + q + 3] = v.w;
                    }
                }
            };
            if (patched) {
                if (DT == 1) {
                    // widen the bf16 tile to fp32 in shared memory so single entries can be rewritten
                    read_raw();
#pragma unroll
                    for (int j = 0; j < NV; ++j) {
                        float *p = conv + warp * WARP_TILE + j * 32 * VEC + lane * VEC;
#pragma unroll
                        for (int q = 0; q < VEC; q += 4)
                            *reinterpret_cast<float4 *>(p + q) = make_float4(e[j * VEC + q], e[j * VEC + q + 1], e[j * VEC + q + 2], e[j * VEC + q + 3]);
                    }
                }
                csync();
                // penalties and biases commute with the mask (a masked logit stays -inf), so they are applied to
                // the unmasked tile and the mask is applied when the lanes read their elements
                bool bad = false;
                auto pen = [&](int id, int ct) {
                    if (id < 0 || id >= P.V) { bad = true; return; }
                    const int li = id - tile_base;
                    if (li >= 0 && li < CTA_TILE) ptile[li] = apply_penalties(ptile[li], ct, c);
                };
                if (tid < c.hist_len) pen(h_id0, h_ct0);
                if (tid + STREAM_THREADS < c.hist_len) pen(h_id1, h_ct1);
                for (int t = tid + 2 * STREAM_THREADS; t < c.hist_len; t += STREAM_THREADS) pen(__ldg(hid + t), __ldg(hct + t));
                csync();
                auto add = [&](int id, float v) {
                    if (id < 0 || id >= P.V) { bad = true; return; }
                    const int li = id - tile_base;
                    if (li >= 0 && li < CTA_TILE) ptile[li] = __fadd_rn(ptile[li], v);
                };
                if (tid < c.bias_len) add(b_id0, b_v0);
                for (int t = tid + STREAM_THREADS; t < c.bias_len; t += STREAM_THREADS) add(__ldg(bid + t), __ldg(bvl + t));
                if (bad && tile == 0) atomicOr(&rs->status, ST_BADID);
                csync();
                read_f32(ptile);
            } else {
                read_raw();
            }
            if (masked && !tail) {
                // the common masked case: one select per element, no bounds test
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const uint32_t bits = __shfl_sync(0xFFFFFFFFu, mword, (j * 32 * VEC + lane * VEC) >> 5) >> ((lane * VEC) & 31);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) e[j * VEC + q] = (bits & (1u << q)) ? e[j * VEC + q] : -CUDART_INF_F;
                }
            } else if (tail) {
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int first = wbase + j * 32 * VEC + lane * VEC;
                    const uint32_t bits = __shfl_sync(0xFFFFFFFFu, mword, (j * 32 * VEC + lane * VEC) >> 5) >> (first & 31);
#pragma unroll
                    for (int q = 0; q < VEC; ++q) {
                        const bool dead = (first + q >= P.V) || (masked && !((bits >> q) & 1u));
                        if (dead) e[j * VEC + q] = -CUDART_INF_F;
                    }
                }
            }
            if (c.div_all) {
#pragma unroll
                for (int q = 0; q < EPL; ++q) e[q] = __fdiv_rn(e[q], c.tau);
            }

            // per-vector maxima, half maxima, lane maximum
            float mv[NV];
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                float m = e[j * VEC];
#pragma unroll
                for (int q = 1; q < VEC; ++q) m = fmaxf(m, e[j * VEC + q]);
                mv[j] = m;
            }
            float h0 = mv[0], h1 = mv[NV / 2];
#pragma unroll
            for (int j = 1; j < NV / 2; ++j) { h0 = fmaxf(h0, mv[j]); h1 = fmaxf(h1, mv[NV / 2 + j]); }
            const float lm = fmaxf(h0, h1);

            if (c.cls == CLS_GREEDY) {
                float wm = lm;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xFFFFFFFFu, wm, off));
                unsigned long long key = 0ull;
                if (wm > -CUDART_INF_F) {
                    int best = 0x7FFFFFFF;
                    if (lm == wm) {
#pragma unroll
                        for (int q = EPL - 1; q >= 0; --q)
                            if (e[q] == wm) best = slot_index<DT>(wbase, lane, q);   // slots ascend: the last write is the lowest
                    }
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) best = min(best, __shfl_xor_sync(0xFFFFFFFFu, best, off));
                    key = ((unsigned long long)okey(wm) << 32) | (uint32_t)(~(uint32_t)best);
                }
                if (lane == 0) sh.best[s][warp] = key;
                csync();
                if (tid == 0) {
                    unsigned long long b = sh.best[s][0];
#pragma unroll
                    for (int w = 1; w < STREAM_WARPS; ++w) b = max(b, sh.best[s][w]);
                    rec->best = b;
                }
            } else {
                // tile cutoff: minimum over G groups of the group maximum, then the largest over the eight warp tiles
                float g;
                const int G = c.G;
                if (G == 0) {
                    g = -CUDART_INF_F;
                } else {
                    const int L = (G >= 32) ? 1 : (32 / G);           // lanes per group
                    g = (G == 64) ? fminf(h0, h1) : lm;
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const float o = __shfl_xor_sync(0xFFFFFFFFu, g, off);
                        g = (off < L) ? fmaxf(g, o) : fminf(g, o);
                    }
                }
                if (lane == 0) sh.tw[s][warp] = g;
                if (tid == 0) sh.ncand[s] = 0;
                csync();
                float t = sh.tw[s][0];
#pragma unroll
                for (int w = 1; w < STREAM_WARPS; ++w) t = fmaxf(t, sh.tw[s][w]);
                // every finite element >= t goes to the tile's candidate slot; a warp reserves its share of the
                // slot with one shared-memory atomic and adds it to the tile record (no second barrier)
                int cnt = 0;
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    if (mv[j] >= t) {
#pragma unroll
                        for (int q = 0; q < VEC; ++q) cnt += (e[j * VEC + q] >= t && e[j * VEC + q] > -CUDART_INF_F) ? 1 : 0;
                    }
                }
                int incl = cnt;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                    if (lane >= off) incl += o;
                }
                const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
                unsigned int base = 0;
                if (lane == 0 && total > 0) {
                    base = atomicAdd(&sh.ncand[s], (unsigned int)total);
                    atomicAdd(&rec->cnt, (unsigned int)total);          // zero before the call; the merge kernel clears it
                }
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
                const int cap_t = (int)(CAND_CAP / (unsigned)tiles);
                if (cnt > 0 && (int)base + total <= cap_t) {
                    unsigned long long *dst = P.cand + (size_t)row * CAND_CAP + (size_t)tile * cap_t + base + (incl - cnt);
#pragma unroll
                    for (int j = 0; j < NV; ++j) {
                        if (mv[j] >= t) {
#pragma unroll
                            for (int q = 0; q < VEC; ++q) {
                                const float v = e[j * VEC + q];
                                if (v >= t && v > -CUDART_INF_F) {
                                    const int idx = slot_index<DT>(wbase, lane, j * VEC + q);
                                    *dst++ = ((unsigned long long)okey(v) << 32) | (uint32_t)(~(uint32_t)idx);
                                }
                            }
                        }
                    }
                }
                if (tid == 0) rec->tkey = okey(t);
            }

            // generic-proxy writes into the stage (in-place patches) precede the next bulk copy into it
            if (DT == 0 && patched) fence_async_proxy();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.empty[s]);
    }
}

// One CTA per row of the streaming classes: combines the tile records and
// finishes the row (global top-k, truncation epilogue, token selection, or the
// per-position verification result).  Rows it cannot prove are flagged for the
// exact kernel.
__global__ void __launch_bounds__(MERGE_THREADS)
sonic_merge_kernel(const KParams P, const int tiles) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ MergeShared<MERGE_THREADS> s_merge;
    const int row = blockIdx.x;
    const int tid = threadIdx.x;
    pdl_launch_dependents();                   // the exact kernel may start on the rows that are its own by class
    const RowCfg c = load_cfg(P, row);         // inputs only: independent of the streaming kernel
    if (c.cls == CLS_EXACT) return;
    pdl_wait_primary();                        // tile records and candidates of the streaming kernel
    RowState *rs = P.rs + row;
    const TileRec *recs = P.tiles + (size_t)row * MAX_TILES;
    const unsigned int status = rs->status;
    if (c.bad || (status & ST_BADID)) {
        if (tid < tiles) P.tiles[(size_t)row * MAX_TILES + tid].cnt = 0u;      // leave the tile counts clean
        if (tid == 0) { emit_row(P, c, row, -1, 0.0f, F_BADPARAM, 0, 0.0f); rs->status = 0; }
        return;
    }
    if (c.cls == CLS_GREEDY) {
        if (tid < 32) {
            unsigned long long best = (tid < tiles) ? recs[tid].best : 0ull;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xFFFFFFFFu, best, off));
            if (tid == 0) {
                if (P.op == OP_TOPK) {
                    // k == 1: a row of nothing but -inf still has a first element
                    P.out_vals[row] = best ? unkey((uint32_t)(best >> 32)) : -CUDART_INF_F;
                    P.out_idx[row] = best ? (int)(~(uint32_t)best) : 0;
                } else if (best == 0ull) {
                    emit_row(P, c, row, -1, 0.0f, F_NO_TOKEN, 0, 0.0f);
                } else {
                    const int token = (int)(~(uint32_t)best);
                    uint32_t flags = 0;
                    float pd = 0.0f;
                    if (P.op == OP_VERIFY && c.l < P.K) {
                        const bool acc = P.draft_tokens[(size_t)c.b * P.K + c.l] == token;
                        if (acc) { flags |= F_ACCEPT; pd = 1.0f; }
                    }
                    emit_row(P, c, row, token, 1.0f, flags, 1, pd);
                }
            }
        }
        return;
    }
    const bool ok = merge_topk_row<MERGE_THREADS, BlockSync>(P, c, row, tiles, reinterpret_cast<unsigned long long *>(smem_raw), s_merge, tid);
    if (tid == 0 && !ok) rs->status = ST_FAILED;
}

}  // namespace sonic
