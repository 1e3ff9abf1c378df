// Streaming kernel and merge kernel.
//
// The streaming kernel reads every logit of the rows of the streaming classes
// exactly once, applies the logit-processing prologue, and reduces each
// 8192-element tile either to an argmax (greedy rows) or to the complete set of
// elements at or above a tile cutoff (top-k rows), written to the tile's own
// slot of the workspace.  The merge kernel, a programmatic dependent launch with
// one CTA per row, combines a row's tile records and finishes the row (global
// top-k, truncation epilogue, token selection) or flags it for the exact kernel.
// The two correspond to the paper's Algorithms "Stage 1: Tile-Local Reduction
// Kernel" and "Stage 2: Cross-Tile Merge and Selection Kernel"; the selection
// itself is ours.
//
// Structure of the streaming kernel: persistent CTAs (three per SM), each a
// producer warp plus eight consumer warps.  The producer takes tiles from a work
// queue, resolves each tile's row configuration and issues one bulk-TMA copy
// (cp.async.bulk, completion on an mbarrier) of the tile's logits into a ring of
// two shared-memory stages, one tile ahead of the consumers, so HBM requests
// stay in flight while the consumers compute.  Every mbarrier wait is bounded:
// on expiry the kernel records an error in the workspace header and returns.
//
// Exactness: a tile's cutoff t is a minimum of group maxima (of the G groups of
// one warp tile, or of all 8 G groups of the tile), so the tile holds elements
// >= t, and it emits EVERY finite element >= t.  With T the largest cutoff of
// the row, the emitted elements >= T are exactly the row's elements >= T.  If
// there are at least k of them the row's top-k is their top-k; otherwise the row
// is handed to the exact kernel.
#pragma once
#include "sonic_common.cuh"
#include "sonic_dense.cuh"

namespace sonic {

template <int DT> struct VecTraits;
template <> struct VecTraits<0> { static constexpr int VEC = 4, NV = 8, NSTAGE = 2, ELT = 4; };
template <> struct VecTraits<1> { static constexpr int VEC = 8, NV = 4, NSTAGE = 2, ELT = 2; };

constexpr int STREAM_CTA_THREADS = STREAM_THREADS + 32;      // eight consumer warps + the producer warp
#ifndef SONIC_WAIT_LIMIT
#define SONIC_WAIT_LIMIT (1u << 22)
#endif
constexpr unsigned int WAIT_LIMIT = SONIC_WAIT_LIMIT;        // try_wait rounds before a wait gives up (a test-only build shortens it)

// ---------------------------------------------------------------- mbarrier / bulk-copy primitives
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Announces `bytes` of a copy to the barrier's current phase without arriving on it (the arrival follows later).
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, unsigned int bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
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
// One bulk copy global -> this CTA's shared memory; bytes and both addresses are multiples of 16.  The logits are
// read once, so the copy carries an evict-first L2 policy: the stream does not push the workspace (candidates,
// tile records) and the kernels' code out of L2.
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_load(void *dst, const void *src, unsigned int bytes, unsigned long long *bar,
                                          unsigned long long policy) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)), "l"(policy) : "memory");
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
    int wsum[THREADS / 32];                    // a block scan's warp totals
    int bracket[4];                            // the counting bins' answer: bin, count above it, count with it
    alignas(16) double scratch[THREADS];      // also read as int4
};


constexpr int RANK_SORT_MAX = 512;            // at most this many candidates: sort by rank counting
constexpr int WARP_EPILOGUE_MAX = 128;        // at most this many survivors of TopK: one warp finishes the row
struct WarpSync { __device__ __forceinline__ void operator()() const { __syncwarp(); } };

template <int NT, typename Sync, typename SH>
__device__ void merge_epilogue(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells);
template <int THREADS, typename SH>
__device__ void merge_epilogue_small(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells);

// Row merge for top-k class rows (one CTA per row).  buf is MERGE_CAP 64-bit
// words of shared memory.  Returns false if the candidates cannot prove the
// row's answer.
template <int THREADS, typename Sync>
__device__ bool merge_topk_row(const KParams &P, const RowCfg &c, int row, int tiles,
                               unsigned long long *buf, MergeShared<THREADS> &sh, int tid, uint2 cells) {
    Sync csync;
    const int cap_t = (int)(P.cand_stride / (unsigned)tiles);
    const TileRec *rec = P.tiles + (size_t)row * MAX_TILES;
    // tile records: the first warp takes one tile per lane; prefix of the counts and the largest cutoff by shuffles
    static_assert(MAX_TILES <= 32, "one tile record per lane of the first warp");
    if (tid < 32) {
        unsigned int cnt = 0u, tk = 0u;
        if (tid < tiles) {
            cnt = __ldcg(&rec[tid].cnt);
            tk = __ldcg(&rec[tid].tkey);
        }
        const bool over = __any_sync(0xFFFFFFFFu, cnt > (unsigned int)cap_t);     // a tile overflowed its slot
        int incl = (int)cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (tid >= off) incl += o;
        }
        tk = __reduce_max_sync(0xFFFFFFFFu, tk);
        sh.tcnt[tid + 1] = incl;                                   // lanes past the last tile repeat the total
        if (tid == 0) { sh.tcnt[0] = 0; sh.count = 0; sh.tkey = tk; sh.found = over ? 1 : 0; }
    }
    csync();
    if (sh.found) return false;
    const unsigned int tkey = sh.tkey;
    const bool complete = (tkey == KEY_NEG_INF);
    const bool strict = c.temp && !complete;            // keys are compared after the temperature division
    const uint32_t tykey = c.temp ? okey(div_tau(unkey(tkey), c.tau)) : tkey;
    const int total = sh.tcnt[tiles];
    // candidates are fetched eight per lane at a time (independent loads), then filtered and packed
    constexpr int GB = 8;
    // proven candidate -> its key after the temperature division (0 if it is not proven)
    auto proven_key = [&](unsigned long long cd, int j) -> unsigned long long {
        const uint32_t zk = (uint32_t)(cd >> 32);
        uint32_t yk = zk;
        if (c.temp) yk = okey(div_tau(unkey(zk), c.tau));
        const bool keep = (j < total) && (zk >= tkey) && !(strict && yk <= tykey);
        return keep ? (((unsigned long long)yk << 32) | (uint32_t)cd) : 0ull;
    };
    unsigned long long floor_key = 1ull;           // keys below it are left out (1: every proven candidate)
    // Large k: while the candidates are gathered they are also counted in 1024 bins of 8192 keys above the proven
    // threshold (one binade of fp32 keys; whatever lies higher shares the top bin).  The bin in which the count from
    // the top reaches k then brackets the k-th key without a pass of its own (GBINS ints in sh.scratch).
    constexpr int GBINS = 2 * THREADS, GSHIFT = 13;
    static_assert(GBINS * 4 <= THREADS * 8, "the counting bins live in the scratch words");
    int *ghist = reinterpret_cast<int *>(sh.scratch);
    const uint32_t gbase = c.temp ? tykey : tkey;
    const bool use_bins = !complete && c.k > RANK_SORT_MAX / 2 && total > RANK_SORT_MAX;
    auto gbin = [&](unsigned long long key) -> int {
        const uint32_t d = ((uint32_t)(key >> 32) - gbase) >> GSHIFT;
        return (int)min(d, (uint32_t)(GBINS - 1));
    };
    // the bin in which the count from the top reaches `need`, the count above it and the count with it (bin < 0: the
    // bins hold fewer than `need`); thread t owns bins GBINS-1-2t and GBINS-2-2t.  Two barriers.
    auto bins_find = [&](int need, int &bin, int &above, int &with) {
        constexpr int BPT = GBINS / THREADS;
        const int lane_ = tid & 31, warp_ = tid >> 5;
        int v[BPT], sum = 0;
#pragma unroll
        for (int j = 0; j < BPT; ++j) { v[j] = ghist[GBINS - 1 - (tid * BPT + j)]; sum += v[j]; }
        int incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane_ >= off) incl += o;
        }
        if (lane_ == 31) sh.wsum[warp_] = incl;
        if (tid == 0) sh.bracket[0] = -1;
        csync();
        int pre = incl - sum;
        for (int w = 0; w < warp_; ++w) pre += sh.wsum[w];
        if (pre < need && pre + sum >= need) {
            int run = pre;
#pragma unroll
            for (int j = 0; j < BPT; ++j) {
                if (run < need && run + v[j] >= need) { sh.bracket[0] = GBINS - 1 - (tid * BPT + j); sh.bracket[1] = run; sh.bracket[2] = run + v[j]; }
                run += v[j];
            }
        }
        csync();
        bin = sh.bracket[0]; above = sh.bracket[1]; with = sh.bracket[2];
        csync();
    };
    for (int attempt = 0; attempt < 2; ++attempt) {
        unsigned long long kmax = 0ull;
        if (use_bins) {
            for (int i = tid; i < GBINS; i += THREADS) ghist[i] = 0;
            csync();
        }
        // tile-major: a warp takes tiles w and w + NW together, its lanes the slots' entries (no search for the
        // tile of an entry; the loads of both tiles are in flight at once)
        constexpr int NW = THREADS / 32, HB = GB / 2;
        const int lane = tid & 31, warp = tid >> 5;
        for (int ta = warp; ta < tiles; ta += 2 * NW) {
            const int tb = ta + NW;
            const int na = sh.tcnt[ta + 1] - sh.tcnt[ta];
            const int nb = (tb < tiles) ? sh.tcnt[tb + 1] - sh.tcnt[tb] : 0;
            const bool single = tb >= tiles;            // no second tile for this warp: all load slots go to the first
            const unsigned long long *pa = P.cand + (size_t)row * P.cand_stride + (size_t)ta * cap_t;
            const unsigned long long *pb = P.cand + (size_t)row * P.cand_stride + (size_t)tb * cap_t;
            if (max(na, nb) <= 32) {
                // small k: a tile brings a dozen candidates, one per lane
                const unsigned long long ca = (lane < na) ? __ldcg(pa + lane) : 0ull;
                const unsigned long long cb = (lane < nb) ? __ldcg(pb + lane) : 0ull;
                const unsigned long long oa = proven_key(ca, lane < na ? 0 : total);
                const unsigned long long ob = proven_key(cb, lane < nb ? 0 : total);
                kmax = max(kmax, max(oa, ob));
                const unsigned int ma = __ballot_sync(0xFFFFFFFFu, oa >= floor_key);
                const unsigned int mb = __ballot_sync(0xFFFFFFFFu, ob >= floor_key);
                const int nk = __popc(ma) + __popc(mb);
                int base = 0;
                if (lane == 0 && nk) base = atomicAdd(&sh.count, nk);
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
                const unsigned int below = (1u << lane) - 1u;
                if (oa >= floor_key) { const int pos = base + __popc(ma & below); if (pos < MERGE_CAP) buf[pos] = oa; if (use_bins) atomicAdd(&ghist[gbin(oa)], 1); }
                if (ob >= floor_key) { const int pos = base + __popc(ma) + __popc(mb & below); if (pos < MERGE_CAP) buf[pos] = ob; if (use_bins) atomicAdd(&ghist[gbin(ob)], 1); }
                continue;
            }
            for (int j0 = 0; j0 < max(na, nb); j0 += (single ? 32 * GB : 32 * HB)) {
                unsigned long long cd[GB];
#pragma unroll
                for (int u = 0; u < HB; ++u) {
                    const int j = j0 + u * 32 + lane, j2 = j + 32 * HB;
                    cd[u] = (j < na) ? __ldcg(pa + j) : 0ull;
                    cd[HB + u] = single ? ((j2 < na) ? __ldcg(pa + j2) : 0ull) : ((j < nb) ? __ldcg(pb + j) : 0ull);
                }
                // filter all of the batch, then reserve room with ONE shared-memory atomic per warp and batch
                // (every warp adds to the same counter: per-candidate or per-slot atomics would queue up there)
                unsigned long long out[GB];
                unsigned int km[GB];
                int nkeep = 0;
#pragma unroll
                for (int u = 0; u < GB; ++u) {
                    const int j = j0 + (u % HB) * 32 + lane + ((single && u >= HB) ? 32 * HB : 0);
                    const bool valid = (u < HB || single) ? (j < na) : (j < nb);
                    out[u] = proven_key(cd[u], valid ? 0 : total);
                    kmax = max(kmax, out[u]);
                    km[u] = __ballot_sync(0xFFFFFFFFu, out[u] >= floor_key);
                    nkeep += __popc(km[u]);
                }
                int base = 0;
                if (lane == 0 && nkeep) base = atomicAdd(&sh.count, nkeep);
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
#pragma unroll
                for (int u = 0; u < GB; ++u) {
                    if (out[u] >= floor_key) {
                        const int pos = base + __popc(km[u] & ((1u << lane) - 1u));
                        if (pos < MERGE_CAP) buf[pos] = out[u];
                        if (use_bins) atomicAdd(&ghist[gbin(out[u])], 1);
                    }
                    base += __popc(km[u]);
                }
            }
        }
        csync();
        if (attempt == 1 || sh.count <= MERGE_CAP || sh.count < c.k) break;
        // More proven candidates than the buffer holds (large k): a key floor that keeps between k and MERGE_CAP of
        // them, then pack again.  The bins counted during the pass usually give it at once ...
        if (use_bins) {
            int b, above, with;
            bins_find(c.k, b, above, with);
            if (b >= 0 && with <= MERGE_CAP) {
                floor_key = max(1ull, ((unsigned long long)gbase + ((unsigned long long)b << GSHIFT)) << 32);
                if (tid == 0) sh.count = 0;
                csync();
                continue;
            }
        }
        // ... otherwise a counting pass over the candidates in global memory, and an eight-way search if that leaves too many.
        unsigned long long *red = reinterpret_cast<unsigned long long *>(sh.scratch);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, off));
        if ((tid & 31) == 0) red[tid >> 5] = kmax;
        csync();
        for (int w = 0; w < THREADS / 32; ++w) kmax = max(kmax, red[w]);
        csync();
        // every proven key is at least (cutoff key << 32): the search starts from the range the keys can span
        unsigned long long lo = max(1ull, (unsigned long long)(c.temp ? tykey : tkey) << 32), hi = kmax + 1ull;   // count(>= lo) >= k > count(>= hi) = 0
        bool bracketed = false;
        {
            // First a bracket from one counting pass: 2048 bins over the keys the proven candidates span, counted from
            // the top; the bin in which the count reaches k gives a floor that keeps at least k, and usually no more
            // than the buffer holds (the search below then has nothing left to do).
            int *hist = reinterpret_cast<int *>(buf);            // (what was packed so far is dropped: it is packed again below)
            int *redi = reinterpret_cast<int *>(sh.scratch);
            const uint32_t klo = (uint32_t)(lo >> 32), khi = (uint32_t)(kmax >> 32);
            const uint32_t span = khi - klo;
            const int shift = span < 2048u ? 0 : (32 - __clz(span)) - 11;
            for (int i = tid; i < 2048; i += THREADS) hist[i] = 0;
            csync();
            for (int ta = warp; ta < tiles; ta += 2 * NW) {
                const int tb = ta + NW;
                const int na = sh.tcnt[ta + 1] - sh.tcnt[ta];
                const int nb = (tb < tiles) ? sh.tcnt[tb + 1] - sh.tcnt[tb] : 0;
                const bool single = tb >= tiles;            // no second tile for this warp: all load slots go to the first
                const unsigned long long *pa = P.cand + (size_t)row * P.cand_stride + (size_t)ta * cap_t;
                const unsigned long long *pb = P.cand + (size_t)row * P.cand_stride + (size_t)tb * cap_t;
                for (int j0 = 0; j0 < max(na, nb); j0 += (single ? 32 * GB : 32 * HB)) {
                    unsigned long long cd[GB];
#pragma unroll
                    for (int u = 0; u < HB; ++u) {
                        const int j = j0 + u * 32 + lane, j2 = j + 32 * HB;
                        cd[u] = (j < na) ? __ldcg(pa + j) : 0ull;
                        cd[HB + u] = single ? ((j2 < na) ? __ldcg(pa + j2) : 0ull) : ((j < nb) ? __ldcg(pb + j) : 0ull);
                    }
#pragma unroll
                    for (int u = 0; u < GB; ++u) {
                        const int j = j0 + (u % HB) * 32 + lane + ((single && u >= HB) ? 32 * HB : 0);
                        const bool valid = (u < HB || single) ? (j < na) : (j < nb);
                        const unsigned long long out = proven_key(cd[u], valid ? 0 : total);
                        if (out >= lo) atomicAdd(&hist[(khi - (uint32_t)(out >> 32)) >> shift], 1);
                    }
                }
            }
            csync();
            static_assert(2048 % THREADS == 0, "bins per thread");
            constexpr int BPT = 2048 / THREADS;
            int v[BPT], s = 0;
#pragma unroll
            for (int j = 0; j < BPT; ++j) { v[j] = hist[tid * BPT + j]; s += v[j]; }
            int incl = s;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += o;
            }
            if (lane == 31) redi[warp] = incl;
            if (tid == 0) redi[40] = -1;
            csync();
            int pre = incl - s;
            for (int w = 0; w < warp; ++w) pre += redi[w];
            if (pre < c.k && pre + s >= c.k) {
                int run = pre;
#pragma unroll
                for (int j = 0; j < BPT; ++j) {
                    if (run < c.k && run + v[j] >= c.k) { redi[40] = tid * BPT + j; redi[41] = run; redi[42] = run + v[j]; }
                    run += v[j];
                }
            }
            csync();
            const int b = redi[40], above = redi[41], kept = redi[42];
            csync();
            if (b >= 0) {
                // bin b holds the keys khi - ((b + 1) << shift) + 1 .. khi - (b << shift)
                const unsigned long long width = 1ull << shift;
                const unsigned long long down = (unsigned long long)(b + 1) * width - 1ull;
                const uint32_t kb = (down >= (unsigned long long)span) ? klo : khi - (uint32_t)down;
                lo = max(lo, (unsigned long long)kb << 32);                                    // count(>= lo) = kept >= k
                if (b > 0) hi = ((unsigned long long)(khi - (uint32_t)((unsigned long long)b * width) + 1u)) << 32;   // count(>= hi) = above < k
                (void)above;
                bracketed = kept <= MERGE_CAP;
            }
        }
        for (int it = 0; it < 24 && !bracketed && hi - lo > 1ull; ++it) {
            const unsigned long long step = (hi - lo) >> 3;
            unsigned long long th[7];
#pragma unroll
            for (int q = 0; q < 7; ++q) th[q] = (step > 0) ? lo + step * (q + 1) : min(hi - 1ull, lo + 1ull + q);
            int cnt[7] = {0, 0, 0, 0, 0, 0, 0};
            // one pass over the candidates, tile-major like the packing pass above
            for (int ta = warp; ta < tiles; ta += 2 * NW) {
                const int tb = ta + NW;
                const int na = sh.tcnt[ta + 1] - sh.tcnt[ta];
                const int nb = (tb < tiles) ? sh.tcnt[tb + 1] - sh.tcnt[tb] : 0;
                const bool single = tb >= tiles;            // no second tile for this warp: all load slots go to the first
                const unsigned long long *pa = P.cand + (size_t)row * P.cand_stride + (size_t)ta * cap_t;
                const unsigned long long *pb = P.cand + (size_t)row * P.cand_stride + (size_t)tb * cap_t;
                for (int j0 = 0; j0 < max(na, nb); j0 += (single ? 32 * GB : 32 * HB)) {
                    unsigned long long cd[GB];
#pragma unroll
                    for (int u = 0; u < HB; ++u) {
                        const int j = j0 + u * 32 + lane, j2 = j + 32 * HB;
                        cd[u] = (j < na) ? __ldcg(pa + j) : 0ull;
                        cd[HB + u] = single ? ((j2 < na) ? __ldcg(pa + j2) : 0ull) : ((j < nb) ? __ldcg(pb + j) : 0ull);
                    }
#pragma unroll
                    for (int u = 0; u < GB; ++u) {
                        const int j = j0 + (u % HB) * 32 + lane + ((single && u >= HB) ? 32 * HB : 0);
                        const bool valid = (u < HB || single) ? (j < na) : (j < nb);
                        const unsigned long long out = proven_key(cd[u], valid ? 0 : total);
#pragma unroll
                        for (int q = 0; q < 7; ++q) cnt[q] += (out >= th[q]) ? 1 : 0;
                    }
                }
            }
            int *redi = reinterpret_cast<int *>(sh.scratch);
#pragma unroll
            for (int q = 0; q < 7; ++q) {
                cnt[q] = (int)__reduce_add_sync(0xFFFFFFFFu, (unsigned int)cnt[q]);
                if ((tid & 31) == 0) redi[(tid >> 5) * 8 + q] = cnt[q];
            }
            csync();
            bool done = false;
            bool fits = false;
            int tots[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
            for (int w = 0; w < THREADS / 32; ++w) {
                const int4 a4 = reinterpret_cast<const int4 *>(redi)[w * 2], b4 = reinterpret_cast<const int4 *>(redi)[w * 2 + 1];
                tots[0] += a4.x; tots[1] += a4.y; tots[2] += a4.z; tots[3] += a4.w;
                tots[4] += b4.x; tots[5] += b4.y; tots[6] += b4.z; tots[7] += b4.w;
            }
#pragma unroll
            for (int q = 6; q >= 0; --q) {                 // the highest threshold that still keeps k
                const int tot = tots[q];
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
    if (Pn > MERGE_CAP) return false;
    int n;
    if (Pn >= c.k) n = c.k;
    else if (complete && P.op != OP_TOPK) n = Pn;
    else return false;
    unsigned long long *sorted = buf;
    int Pn2 = Pn;
    // How many keys the sort below should get at most: what the rank sort takes in one go when n is small, else the
    // bitonic size that leaves the threshold search a window of at least 16 ranks above n (for the largest n the
    // next size up would cost more than searching a narrow window).
    int want_hi = (n + n / 2 + 16 <= RANK_SORT_MAX) ? n + n / 2 + 16 : next_pow2(n + 16);
    if (want_hi > MERGE_CAP / 2) want_hi = next_pow2(n);
    if (Pn > RANK_SORT_MAX && Pn > want_hi) {
        // more proven candidates than that: search a key threshold that keeps between n and want_hi of them (any
        // such threshold keeps the n best), then sort only those
        unsigned long long lo = 0ull, hi = ~0ull;          // count(>= lo) >= n > count(>= hi)
        bool tight = false;
        bool bracketed = false;
        int cnt_lo = Pn, cnt_hi = 0;
        if (use_bins) {
            int b, above, with;
            bins_find(n, b, above, with);
            if (b >= 0) {
                // bin b holds the keys gbase + (b << GSHIFT) .. gbase + ((b + 1) << GSHIFT) - 1 (the top bin: and all above)
                const unsigned long long klo = (unsigned long long)gbase + ((unsigned long long)b << GSHIFT);
                lo = klo << 32;
                hi = (b == GBINS - 1 || klo + (1ull << GSHIFT) > 0xFFFFFFFFull) ? ~0ull : ((klo + (1ull << GSHIFT)) << 32);
                cnt_hi = above;
                cnt_lo = with;
                bracketed = true;
            }
        }
        if (!bracketed) {
            // First bracket from the data itself: 31 of the keys, sorted, split the candidates into 32 buckets of
            // about equal population wherever the keys crowd; one counting pass then places n within one bucket.
            unsigned long long *sth = reinterpret_cast<unsigned long long *>(sh.scratch);          // [32] ascending, last = sentinel
            int *hist = reinterpret_cast<int *>(sh.scratch + 32);                                  // [32]
            unsigned long long *res = reinterpret_cast<unsigned long long *>(sh.scratch + 64);     // lo, hi, count(>= lo), count(>= hi)
            if (tid < 32) {
                unsigned long long k = (tid < 31) ? buf[(int)(((long long)(tid + 1) * Pn) >> 5)] : ~0ull;
#pragma unroll
                for (int kk = 2; kk <= 32; kk <<= 1) {
#pragma unroll
                    for (int jj = kk >> 1; jj > 0; jj >>= 1) {
                        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, k, jj);
                        const bool take_min = (((tid & kk) == 0) == ((tid & jj) == 0));
                        k = ((k < o) == take_min) ? k : o;
                    }
                }
                sth[tid] = k;
                hist[tid] = 0;
            }
            csync();
            for (int i = tid; i < Pn; i += THREADS) {
                const unsigned long long key = buf[i];
                int bkt = 0;                                   // number of sampled keys <= key
#pragma unroll
                for (int step = 16; step > 0; step >>= 1)
                    if (bkt + step <= 31 && sth[bkt + step - 1] <= key) bkt += step;
                atomicAdd(&hist[bkt], 1);
            }
            csync();
            if (tid < 32) {
                int suf = hist[tid];                           // -> number of keys in buckets >= tid
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int dn = __shfl_down_sync(0xFFFFFFFFu, suf, o);
                    if (tid + o < 32) suf += dn;
                }
                // keys >= sth[q] are those of buckets q + 1 and above: the largest such q that still keeps n
                const unsigned int okm = __ballot_sync(0xFFFFFFFFu, tid >= 1 && suf >= n);
                if (okm) {
                    const int l = 31 - __clz(okm);
                    const int cnt = __shfl_sync(0xFFFFFFFFu, suf, l);
                    const int above = (l < 31) ? __shfl_sync(0xFFFFFFFFu, suf, (l + 1) & 31) : 0;     // keys >= hi
                    if (tid == 0) { res[0] = sth[l - 1]; res[1] = sth[l]; res[2] = (unsigned long long)cnt; res[3] = (unsigned long long)above; }
                } else {
                    const int above = __shfl_sync(0xFFFFFFFFu, suf, 1);
                    if (tid == 0) { res[0] = 0ull; res[1] = sth[0]; res[2] = (unsigned long long)Pn; res[3] = (unsigned long long)above; }
                }
            }
            csync();
            lo = res[0]; hi = res[1];
            cnt_lo = (int)res[2]; cnt_hi = (int)res[3];
            csync();
        }
        {
            tight = cnt_lo <= want_hi;
            // The bucket [lo, hi) holds the boundary.  If it is small, its keys are collected and ranked, which gives
            // the threshold that keeps exactly n (no search over key space, whose passes multiply when equal values
            // differ only in their index bits).
            const int in_bucket = cnt_lo - cnt_hi, need_here = n - cnt_hi;         // 1 <= need_here <= in_bucket
            if (!tight && in_bucket <= THREADS) {
                unsigned long long *list = reinterpret_cast<unsigned long long *>(sh.scratch);         // [THREADS]
                if (tid == 0) sh.count = 0;
                csync();
                for (int i0 = 0; i0 < Pn; i0 += THREADS) {
                    const int i = i0 + tid;
                    const unsigned long long key = (i < Pn) ? buf[i] : 0ull;
                    const bool inb = (i < Pn) && key >= lo && key < hi;
                    const unsigned int mk = __ballot_sync(0xFFFFFFFFu, inb);
                    int base = 0;
                    if ((tid & 31) == 0 && mk) base = atomicAdd(&sh.count, __popc(mk));
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    if (inb) list[base + __popc(mk & ((1u << (tid & 31)) - 1u))] = key;
                }
                csync();
                int rank;
                const unsigned long long key = rank_keys<THREADS, Sync>(list, in_bucket, tid, rank);
                csync();
                if (key != 0ull && rank == need_here - 1) list[0] = key;      // exactly one thread (keys are distinct)
                csync();
                lo = list[0];
                tight = true;                                   // count(>= lo) == n
                csync();
            }
        }
        // eight-way search: seven interior thresholds per pass.  The warps add their counts into one of two sets
        // of totals in shared memory (the other set is cleared meanwhile), so a pass costs two block barriers
        // and every thread reads just the seven totals.
        int *tot2 = reinterpret_cast<int *>(sh.scratch);          // [2][8]
        if (tid < 16) tot2[tid] = 0;
        csync();
        int pass = 0;
        for (int it = 0; it < 24 && !tight && hi - lo > 1ull; ++it, ++pass) {
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
            int *tot = tot2 + (pass & 1) * 8;
#pragma unroll
            for (int q = 0; q < 7; ++q) {
                cnt[q] = (int)__reduce_add_sync(0xFFFFFFFFu, (unsigned int)cnt[q]);
                if ((tid & 31) == 0 && cnt[q]) atomicAdd(&tot[q], cnt[q]);
            }
            if (tid < 8) tot2[((pass + 1) & 1) * 8 + tid] = 0;     // the next pass's set (last read before the previous barrier)
            csync();
            const int4 a4 = reinterpret_cast<const int4 *>(tot)[0], b4 = reinterpret_cast<const int4 *>(tot)[1];
            const int tots[7] = {a4.x, a4.y, a4.z, a4.w, b4.x, b4.y, b4.z};
            bool done = false;
#pragma unroll
            for (int q = 6; q >= 0; --q) {                 // the highest threshold that still keeps n
                if (!done && tots[q] >= n) {
                    lo = th[q];
                    if (q < 6) hi = th[q + 1];
                    done = true;
                    if (tots[q] <= want_hi) it = 1000;      // tight enough
                }
            }
            if (!done) hi = th[0];
            csync();
        }
        // keep the keys >= lo, packed to the front
        if (tid == 0) sh.count = 0;
        csync();
        if (Pn <= MERGE_CAP / 2) {
            // room for a copy: pack into the upper half without barriers, then move the survivors down
            unsigned long long *up = buf + MERGE_CAP / 2;
            for (int i0 = 0; i0 < Pn; i0 += THREADS) {
                const int i = i0 + tid;
                const unsigned long long key = (i < Pn) ? buf[i] : 0ull;
                const bool keep = (i < Pn) && key >= lo;
                const unsigned int mk = __ballot_sync(0xFFFFFFFFu, keep);
                int base = 0;
                if ((tid & 31) == 0 && mk) base = atomicAdd(&sh.count, __popc(mk));
                base = __shfl_sync(0xFFFFFFFFu, base, 0);
                if (keep) up[base + __popc(mk & ((1u << (tid & 31)) - 1u))] = key;
            }
            csync();
            const int kept = sh.count;
            for (int i = tid; i < kept; i += THREADS) buf[i] = up[i];
        } else {
            // in place (every position written is at or below one already read)
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
        }
        csync();
        Pn2 = sh.count;
        csync();
    }
    const int PnAll = Pn;
    (void)PnAll;
#define Pn Pn2
    if (Pn <= RANK_SORT_MAX) {
        // few candidates, one per thread: every warp sorts its 32 keys with shuffles, then a key's rank is its
        // place in its own run plus, for every other run, the number of keys there above it (a binary search
        // in the sorted run; keys are distinct, 0 pads the last run).  Two block barriers.
        static_assert(RANK_SORT_MAX <= THREADS, "one candidate per thread");
        unsigned long long *dst = buf + MERGE_CAP / 2;
        {
            int rank;
            const unsigned long long key = rank_keys<THREADS, Sync>(buf, Pn, tid, rank);
            if (key != 0ull) dst[rank] = key;
        }
        csync();
        for (int i = tid; i < n; i += THREADS) buf[i] = dst[i];       // only the n best are used from here on
        csync();
    } else {
        const int m = next_pow2(Pn);
        for (int i = Pn + tid; i < m; i += THREADS) buf[i] = 0ull;
        csync();
        bitonic_sort_desc_cta<THREADS>(buf, m, tid);
    }
    (void)sorted;
#undef Pn

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
        merge_epilogue_small<THREADS>(P, c, row, n, buf, sh, tid, cells);
    } else {
        merge_epilogue<THREADS, Sync>(P, c, row, n, buf, sh, tid, cells);
    }
    return true;
}

// Truncation epilogue and token selection over the n best candidates, sorted in
// buf[0, n) (TopK already applied): TopP, MinP, index-order CDF, Philox draw,
// and for verification rows the accept test and the residual.  Three parts:
// the front (weights, cumulative sums, TopP / MinP: linear work), the index
// order of the survivors (quadratic rank counting, or a sort), and the tail
// (linear again).  Large supports run all three on the whole CTA; small ones
// run the linear parts on one warp, without block barriers, and only the
// quadratic part on all threads.
//
// shared-memory layout after the sort (n <= KFAST_SAMPLE = MERGE_CAP / 4):
//   buf[0, n)     sorted keys (value key << 32 | ~index)
//   w             weights exp(y - M) in ranking order
//   cs            cumulative sums (ranking order), later residual / CDF in index order
//   ik            (~index << 32 | ranking position), sorted descending = index ascending
struct EpiView {
    double *w, *cs;
    unsigned long long *ik;
    __device__ explicit EpiView(unsigned long long *buf)
        : w(reinterpret_cast<double *>(buf + KFAST_SAMPLE)), cs(reinterpret_cast<double *>(buf + 2 * KFAST_SAMPLE)),
          ik(buf + 3 * KFAST_SAMPLE) {}
};

// weights of the candidates (all threads of the caller's group)
template <int NT>
__device__ __forceinline__ void epilogue_weights(int n, unsigned long long *buf, int tid) {
    EpiView v(buf);
    const double M = (double)unkey((uint32_t)(buf[0] >> 32));
    for (int j = tid; j < n; j += NT) {
        double y = (double)unkey((uint32_t)(buf[j] >> 32));
        double wj = exp(y - M);
        v.w[j] = wj; v.cs[j] = wj;
    }
}

// cumulative sums and the TopP / MinP cuts; returns the surviving prefix length (also left in sh.n_p)
template <int NT, typename Sync, typename SH>
__device__ __forceinline__ int epilogue_truncate(const RowCfg &c, int n, unsigned long long *buf, SH &sh, int tid) {
    Sync csync;
    EpiView v(buf);
    const double M = (double)unkey((uint32_t)(buf[0] >> 32));
    block_inclusive_scan<NT, Sync>(v.cs, n, sh.scratch, tid);
    const double Z = v.cs[n - 1];
    if (c.z & M_TOP_P) {
        const double target = (double)c.p * Z;
        for (int j = tid; j < n; j += NT)
            if (v.cs[j] >= target && (j == 0 || v.cs[j - 1] < target)) sh.n_p = j + 1;
    }
    if (c.z & M_MIN_P) {
        const double thr = M + log((double)c.theta);
        for (int j = tid; j < n; j += NT) {
            bool in = (double)unkey((uint32_t)(buf[j] >> 32)) >= thr;
            bool prev_in = (j == 0) || ((double)unkey((uint32_t)(buf[j - 1] >> 32)) >= thr);
            if (!in && prev_in) sh.n_m = j;
        }
    }
    csync();
    n = min(n, min(sh.n_p, sh.n_m));
    csync();
    if (tid == 0) sh.n_p = n;
    csync();
    return n;
}

// The same for one warp and n <= WARP_EPILOGUE_MAX, in registers: a lane holds four consecutive weights, the
// cumulative sums come from one shuffle scan, the cuts from votes.  Leaves the surviving prefix length in sh.n_p
// and its total weight in cs[length - 1].
template <typename SH>
__device__ __forceinline__ void epilogue_truncate_warp(const RowCfg &c, int n, unsigned long long *buf, SH &sh, int lane) {
    static_assert(WARP_EPILOGUE_MAX <= 128, "four elements per lane");
    EpiView v(buf);
    const double M = (double)unkey((uint32_t)(buf[0] >> 32));
    double cs[4];
    double run = 0.0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int j = lane * 4 + u;
        run += (j < n) ? v.w[j] : 0.0;
        cs[u] = run;
    }
    double incl = run;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    const double excl = incl - run;
#pragma unroll
    for (int u = 0; u < 4; ++u) cs[u] += excl;
    const double Z = __shfl_sync(0xFFFFFFFFu, incl, 31);
    // first position (ranking order) where a cut falls, from every lane's first hit among its four (4: none)
    auto first_hit = [&](int mine) -> int {
        const unsigned int m = __ballot_sync(0xFFFFFFFFu, mine < 4);
        if (!m) return -1;
        const int l = __ffs(m) - 1;
        return l * 4 + __shfl_sync(0xFFFFFFFFu, mine, l);
    };
    int keep = n;
    if (c.z & M_TOP_P) {
        const double target = (double)c.p * Z;
        int mine = 4;
#pragma unroll
        for (int u = 3; u >= 0; --u) if (lane * 4 + u < n && cs[u] >= target) mine = u;
        const int j = first_hit(mine);
        if (j >= 0) keep = min(keep, j + 1);
    }
    if (c.z & M_MIN_P) {
        const double thr = M + log((double)c.theta);
        int mine = 4;
#pragma unroll
        for (int u = 3; u >= 0; --u) {
            const int j = lane * 4 + u;
            if (j < n && !((double)unkey((uint32_t)(buf[j] >> 32)) >= thr)) mine = u;          // first element below the threshold
        }
        const int j = first_hit(mine);
        if (j >= 0) keep = min(keep, j);
    }
    // total weight of the survivors: the cumulative sum at position keep - 1
    double mine = 0.0;
#pragma unroll
    for (int u = 0; u < 4; ++u) if (((keep - 1) & 3) == u) mine = cs[u];
    const double W = __shfl_sync(0xFFFFFFFFu, mine, (keep - 1) >> 2);
    if (lane == 0) { sh.n_p = keep; v.cs[keep - 1] = W; }     // the tail reads the survivors' total weight from there
    __syncwarp();
}

// survivors in vocabulary-index order
template <int NT, typename Sync>
__device__ __forceinline__ void epilogue_index_order(int n, unsigned long long *buf, int tid) {
    Sync csync;
    EpiView v(buf);
    if (n <= RANK_SORT_MAX) {
        // few survivors: each lands at the number of survivors with a smaller index; S threads share a survivor
        const int S = min(32, max(1, NT / next_pow2(n)));
        for (int j0 = 0; j0 < n; j0 += NT / S) {
            const int j = j0 + tid / S, seg = tid % S;
            const uint32_t mine = (j < n) ? (uint32_t)buf[j] : 0xFFFFFFFFu;      // ~index: larger means smaller index
            const int tlo = (int)(((long long)n * seg) / S), thi = (int)(((long long)n * (seg + 1)) / S);
            int pos = 0;
            int t = tlo;
            for (; t + 8 <= thi; t += 8) {
                uint32_t o[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) o[u] = (uint32_t)buf[t + u];
#pragma unroll
                for (int u = 0; u < 8; ++u) pos += (o[u] > mine) ? 1 : 0;
            }
            for (; t < thi; ++t) pos += ((uint32_t)buf[t] > mine) ? 1 : 0;
            for (int off = 1; off < S; off <<= 1) pos += __shfl_xor_sync(0xFFFFFFFFu, pos, off);
            if (seg == 0 && j < n) v.ik[pos] = ((unsigned long long)mine << 32) | (unsigned long long)j;
        }
        csync();
    } else {
        const int m2 = next_pow2(n);
        for (int j = tid; j < m2; j += NT)
            v.ik[j] = (j < n) ? ((buf[j] << 32) | (unsigned long long)j) : 0ull;
        csync();
        if constexpr (NT >= 64) bitonic_sort_desc_cta<NT>(v.ik, m2, tid);
        else bitonic_sort_desc<NT, Sync>(v.ik, m2, tid);
    }
}

// draw, verification, selection and the row's outputs
template <int NT, typename Sync, typename SH>
__device__ __forceinline__ void epilogue_tail(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells) {
    Sync csync;
    constexpr int THREADS = NT;
    EpiView v(buf);
    double *w = v.w, *cs = v.cs;
    unsigned long long *ik = v.ik;
    const double W = cs[n - 1];                 // still the ranking-order cumulative sums here
    csync();
    const uint32_t a_acc = cells.x, a_draw = cells.y;      // the row's Philox cells, drawn before the wait on the streaming kernel
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
        if (!accept) {        // (an accepted position's own token is never read: the request moves on with the draft)
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
    }
    bool picked = false;
    if constexpr (NT == 32) {
        if (!use_residual) {
            // one warp, at most 128 survivors: the index-order cumulative weights stay in registers (a lane holds
            // four consecutive positions), the drawn position comes from a vote
            double csr[4];
            double run = 0.0;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = tid * 4 + u;
                run += (j < n) ? w[(uint32_t)ik[j]] : 0.0;
                csr[u] = run;
            }
            double incl = run;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (tid >= o) incl += up;
            }
            const double excl = incl - run;
            const double target = u_draw * __shfl_sync(0xFFFFFFFFu, incl, 31);
            int mine = 4;
#pragma unroll
            for (int u = 3; u >= 0; --u) if (tid * 4 + u < n && csr[u] + excl > target) mine = u;
            const unsigned int m = __ballot_sync(0xFFFFFFFFu, mine < 4);
            int j = n - 1;
            if (m) { const int l = __ffs(m) - 1; j = l * 4 + __shfl_sync(0xFFFFFFFFu, mine, l); }
            if (tid == 0) sh.pick = j;
            picked = true;
            __syncwarp();
        }
    }
    if (!picked) {
        if (!use_residual) {
            for (int j = tid; j < n; j += THREADS) cs[j] = w[(uint32_t)ik[j]];
            csync();
            block_inclusive_scan<THREADS, Sync>(cs, n, sh.scratch, tid);
        }
        const double R = cs[n - 1];
        const double target = u_draw * R;
        if (tid == 0) sh.pick = n - 1;
        csync();
        for (int j = tid; j < n; j += THREADS)
            if (cs[j] > target && (j == 0 || !(cs[j - 1] > target))) sh.pick = j;
        csync();
    }
    if (tid == 0) {
        int j = sh.pick;
        int token = (int)(~(uint32_t)(ik[j] >> 32));
        float prob = (float)(w[(uint32_t)ik[j]] / W);
        emit_row(P, c, row, token, prob, flags, n, p_draft);
    }
}


// The draw of a sampling row with a large support (more survivors than the rank counting takes): the survivors are not
// brought into index order at all.  Their weights, as 2^-40 fixed-point integers, are added up per tile, then per 256 ids
// of the tile the target falls into, then per id of that range; each level is one pass over the survivors, a scan of
// at most 256 bins and a barrier.  Integer sums: the same token in every replay; against the exact index-order CDF the
// target moves by less than n * 2^-40 of the mass.
template <int NT, typename Sync, typename SH>
__device__ void epilogue_draw_large(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells) {
    Sync csync;
    static_assert(NT >= 256, "a thread per bin");
    EpiView v(buf);
    const double *w = v.w;
    const double W = v.cs[n - 1];                              // ranking-order cumulative sums: the support's mass
    unsigned int *blo = reinterpret_cast<unsigned int *>(v.ik), *bhi = blo + 256;      // (the index keys' place: unused on this path)
    unsigned long long *red = reinterpret_cast<unsigned long long *>(sh.scratch);
    const int lane = tid & 31, warp = tid >> 5;
    auto fixed = [&](int j) -> unsigned long long { return (unsigned long long)(w[j] * 1099511627776.0); };
    unsigned int range_lo = 0u;
    unsigned long long rest = 0ull;
    const int shifts[3] = {13, 8, 0};
    const unsigned int spans[3] = {(unsigned int)MAX_TILES << 13, 8192u, 256u};
#pragma unroll
    for (int level = 0; level < 3; ++level) {
        const int shift = shifts[level];
        const unsigned int span = spans[level];
        const int nb = (int)(span >> shift);                   // 32, 32, 256
        if (tid < 256) { blo[tid] = 0u; bhi[tid] = 0u; }
        csync();
        for (int j = tid; j < n; j += NT) {
            const unsigned int idx = ~(uint32_t)buf[j];
            const unsigned int d = idx - range_lo;
            const unsigned long long q = fixed(j);
            if (d < span && q) {
                const int b = (int)(d >> shift);
                const unsigned int lo = (unsigned int)q, hi = (unsigned int)(q >> 32);
                unsigned int carry = 0u;
                if (lo) { const unsigned int old = atomicAdd(&blo[b], lo); carry = (old + lo < old) ? 1u : 0u; }
                if (hi + carry) atomicAdd(&bhi[b], hi + carry);
            }
        }
        csync();
        // scan of the bins (a thread per bin, warps in order)
        const unsigned long long mine = (tid < nb) ? (((unsigned long long)bhi[tid] << 32) + blo[tid]) : 0ull;
        unsigned long long incl = mine;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) red[warp] = incl;
        if (tid == 0) sh.pick = -1;
        csync();
        unsigned long long before = 0ull, total = 0ull;
        for (int wq = 0; wq < NT / 32; ++wq) { const unsigned long long t = red[wq]; before += (wq < warp) ? t : 0ull; total += t; }
        if (level == 0) rest = draw_target(total, cells.y);     // the support's mass in fixed point, and the draw's target in it
        const unsigned long long excl = before + incl - mine;
        if (mine > 0ull && excl <= rest && rest < excl + mine) { sh.pick = tid; red[32] = excl; }
        csync();
        int b = sh.pick;
        if (b < 0) {                                           // (rest < total always; kept for safety: the last bin with mass)
            if (mine > 0ull) atomicMax(&sh.pick, tid);
            csync();
            b = sh.pick;
            if (tid == b) red[32] = excl;
            csync();
        }
        const unsigned long long excl_b = red[32];
        rest = (rest > excl_b) ? rest - excl_b : 0ull;
        range_lo += (unsigned int)b << shift;
        csync();
    }
    // the survivor with that id
    if (tid == 0) sh.pick = 0;
    csync();
    for (int j = tid; j < n; j += NT)
        if (~(uint32_t)buf[j] == range_lo) sh.pick = j;
    csync();
    if (tid == 0) {
        const int j = sh.pick;
        emit_row(P, c, row, (int)(~(uint32_t)buf[j]), (float)(w[j] / W), 0u, n, 0.0f);
    }
}

template <int NT, typename Sync, typename SH>
__device__ void merge_epilogue(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells) {
    Sync csync;
    epilogue_weights<NT>(n, buf, tid);
    if (tid == 0) { sh.n_p = n; sh.n_m = n; sh.found = 0; sh.pick = -1; }
    csync();
    n = epilogue_truncate<NT, Sync>(c, n, buf, sh, tid);
    if (P.op == OP_SAMPLE && n > RANK_SORT_MAX) {
        epilogue_draw_large<NT, Sync>(P, c, row, n, buf, sh, tid, cells);
        return;
    }
    epilogue_index_order<NT, Sync>(n, buf, tid);
    epilogue_tail<NT, Sync>(P, c, row, n, buf, sh, tid, cells);
}

// Small supports: the linear parts on warp 0 (warp-level synchronisation only), the weights and the quadratic
// index ranking on the whole CTA.  Three block barriers in all.
template <int THREADS, typename SH>
__device__ void merge_epilogue_small(const KParams &P, const RowCfg &c, int row, int n, unsigned long long *buf, SH &sh, int tid, uint2 cells) {
    epilogue_weights<THREADS>(n, buf, tid);
    if (tid == 0) { sh.n_p = n; sh.n_m = n; sh.found = 0; sh.pick = -1; }
    __syncthreads();
    if (tid < 32) epilogue_truncate_warp(c, n, buf, sh, tid);
    __syncthreads();
    n = sh.n_p;
    epilogue_index_order<THREADS, BlockSync>(n, buf, tid);
    if (tid < 32) epilogue_tail<32, WarpSync>(P, c, row, n, buf, sh, tid, cells);
}

// Smallest of a warp tile's group maxima, L lanes per group (g: the lane's own maximum, or with half-lane groups
// the smaller of its two).  In tile mode a group without a finite element counts as +inf, i.e. takes no part.
template <int L>
__device__ __forceinline__ float warp_cutoff(float g, bool tile_mode) {
#pragma unroll
    for (int off = 1; off < L; off <<= 1) g = fmaxf(g, __shfl_xor_sync(0xFFFFFFFFu, g, off));
    if (tile_mode && g == -CUDART_INF_F) g = CUDART_INF_F;
#pragma unroll
    for (int off = L; off < 32; off <<= 1) g = fminf(g, __shfl_xor_sync(0xFFFFFFFFu, g, off));
    return g;
}

// What the producer hands to the consumers with each stage.
struct StageMeta {
    RowCfg cfg;
    int row, tile;
    int skip;                                  // the row belongs to the exact kernel: nothing was loaded
    int patch;                                 // 0 none, 1 the producer filtered the lists into hits[], 2 consumers scan the lists
    int npen, nbias;                           // hits of this tile
    int hb;                                    // which hit buffer holds them
    int stop;                                  // no more tiles for this CTA (nothing else in the entry is valid)
    int bad;                                   // the producer met a list id outside [0, V)
    int next_row, next_tile;                   // the tile that follows (-1: none, or not known yet)
};
struct Hit { int li; int payload; };           // element within the tile; history count, or the bias as float bits

template <int DT>
struct StreamShared {
    static constexpr int NSTAGE = VecTraits<DT>::NSTAGE;
    unsigned long long full[NSTAGE];           // producer -> consumers: stage described and copy issued (one arrival + the copy's bytes)
    unsigned long long empty[NSTAGE];          // consumers -> producer: stage free (one arrival per consumer warp)
    StageMeta meta[NSTAGE];
    // per-stage scratch of the consumer warps (a fast warp may already be on the next tile, in the other stage)
    alignas(16) float tw[NSTAGE][STREAM_WARPS];
    unsigned int ncand[NSTAGE];
    unsigned long long best[NSTAGE][STREAM_WARPS];
    unsigned int kmin[NSTAGE][STREAM_WARPS], nfin[NSTAGE][STREAM_WARPS];     // dense rows
    // hit lists: one buffer more than stages, so that the producer fills the next tile's while both stages are busy
    Hit pen[NSTAGE + 1][HIT_PEN_CAP];
    Hit bias[NSTAGE + 1][HIT_BIAS_CAP];
};

template <int DT>
__global__ void __launch_bounds__(STREAM_CTA_THREADS, 3)
sonic_stream_kernel(const KParams P, const int tiles, const int nitems, const int chunk, const int cap_t) {     // cap_t: candidate slots per tile, CAND_CAP / tiles
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
    KERNEL_T0(0);
    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], STREAM_WARPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (blockIdx.x == 0 && tid == 0) P.error[WS_FAILED_ROWS] = 0u;     // this call's count of rows the merge kernel cannot prove
    __syncthreads();
    pdl_launch_dependents();                   // the merge kernel may start launching; it waits for this grid to finish

    if (warp == STREAM_WARPS) {
        // ------------------------------------------------------------ producer warp
        // The (row, tile) items are handed out through a counter in the workspace, so CTAs that become resident
        // late (the SMs may be shared with the exact kernel) find less or no work instead of holding back a fixed
        // share.  Per tile the
        // producer (1) waits for a free stage, describes the tile and issues its bulk copy, then (2) prepares
        // the NEXT tile while the ring is busy.  On a new row that means one round of global loads (parameters
        // and sparse lists, kept in registers for the row's other tiles); on every tile, picking the list
        // entries that fall into it and writing them to a hit buffer, so that the consumers patch only what is
        // there, each warp only its own part of the tile.
        static_assert(SONIC_MAX_VOCAB <= (1 << 18), "packed history entries hold an 18-bit id");
        constexpr int HPL = FILTER_HIST / 32;      // packed history entries per lane
        struct Prep { int patch, npen, nbias; };
        int memo_k = -1, memo_G = -1;
        RowCfg c_next;
        uint32_t packed[HPL];                      // id | count << 18; 0 = no entry
        int b_id = -1;
        float b_val = 0.0f;
        int row_patch = 0, cached_row = -1, row_bad = 0;
        auto load_row = [&](int row) {
            const int req = (P.op == OP_VERIFY) ? row / (P.K + 1) : row;
            const int *hid = P.hist_ids ? P.hist_ids + (size_t)req * P.hist_stride : nullptr;
            const int *hct = P.hist_counts ? P.hist_counts + (size_t)req * P.hist_stride : nullptr;
            const int *bid = P.bias_ids ? P.bias_ids + (size_t)req * P.bias_stride : nullptr;
            const float *bvl = P.bias_vals ? P.bias_vals + (size_t)req * P.bias_stride : nullptr;
            // the first round of loads goes out before the first use (the lengths arrive with the parameters:
            // bound by the strides); the second half of a long history follows in a round of its own
            constexpr int HALF = HPL / 2;
            const CfgRaw raw = fetch_cfg(P, row);
            int id[HALF], ct[HALF];
#pragma unroll
            for (int u = 0; u < HALF; ++u) {
                const int t = lane + 32 * u;
                id[u] = -1; ct[u] = 0;
                if (hid && hct && t < P.hist_stride) { id[u] = __ldg(hid + t); ct[u] = __ldg(hct + t); }
            }
            int b0 = -1; float v0 = 0.0f;
            if (bid && bvl && lane < P.bias_stride) { b0 = __ldg(bid + lane); v0 = __ldg(bvl + lane); }
            c_next = resolve_cfg(P, row, raw, &memo_k, &memo_G);
            cached_row = row;
            row_patch = 0;
            row_bad = 0;
            if (c_next.cls == CLS_EXACT || !(c_next.hist_len > 0 || c_next.bias_len > 0)) return;
            row_patch = 2;
            if (c_next.hist_len > FILTER_HIST || c_next.bias_len > FILTER_BIAS) return;
            bool bad = false, big = false;
            auto pack = [&](int t, int i, int cnt) -> uint32_t {
                if (t >= c_next.hist_len) return 0u;
                if (i < 0 || i >= P.V) { bad = true; return 0u; }
                if (cnt > FILTER_COUNT_MAX) { big = true; return 0u; }
                return (cnt > 0) ? ((uint32_t)i | ((uint32_t)cnt << 18)) : 0u;
            };
#pragma unroll
            for (int u = 0; u < HALF; ++u) packed[u] = pack(lane + 32 * u, id[u], ct[u]);
#pragma unroll
            for (int u = 0; u < HALF; ++u) packed[HALF + u] = 0u;
            if (c_next.hist_len > 32 * HALF) {
#pragma unroll
                for (int u = 0; u < HALF; ++u) {
                    const int t = lane + 32 * (HALF + u);
                    id[u] = -1; ct[u] = 0;
                    if (t < c_next.hist_len) { id[u] = __ldg(hid + t); ct[u] = __ldg(hct + t); }
                }
#pragma unroll
                for (int u = 0; u < HALF; ++u) packed[HALF + u] = pack(lane + 32 * (HALF + u), id[u], ct[u]);
            }
            b_id = -1; b_val = 0.0f;
            if (lane < c_next.bias_len) {
                if (b0 < 0 || b0 >= P.V) bad = true;
                else { b_id = b0; b_val = v0; }
            }
            row_bad = __any_sync(0xFFFFFFFFu, bad) ? 1 : 0;
            if (__any_sync(0xFFFFFFFFu, big)) return;          // a count too large to pack: consumers scan
            row_patch = 1;
        };
        auto prepare = [&](int row, int tile, int hb) -> Prep {
            if (row != cached_row) load_row(row);
            Prep r{row_patch, 0, 0};
            if (row_patch != 1) return r;
            const int first = tile * CTA_TILE;
#pragma unroll
            for (int u = 0; u < HPL; ++u) {
                const unsigned int li = (packed[u] & 0x3FFFFu) - (unsigned int)first;
                const bool hit = packed[u] != 0u && li < (unsigned int)CTA_TILE;
                const unsigned int hm = __ballot_sync(0xFFFFFFFFu, hit);
                if (hit) {
                    const int pos = r.npen + __popc(hm & ((1u << lane) - 1u));
                    if (pos < HIT_PEN_CAP) { sh.pen[hb][pos].li = (int)li; sh.pen[hb][pos].payload = (int)(packed[u] >> 18); }
                }
                r.npen += __popc(hm);
            }
            {
                const unsigned int li = (unsigned int)(b_id - first);
                const bool hit = b_id >= 0 && li < (unsigned int)CTA_TILE;
                const unsigned int hm = __ballot_sync(0xFFFFFFFFu, hit);
                if (hit) {
                    const int pos = __popc(hm & ((1u << lane) - 1u));
                    sh.bias[hb][pos].li = (int)li; sh.bias[hb][pos].payload = __float_as_int(b_val);
                }
                r.nbias = __popc(hm);
            }
            if (r.npen > HIT_PEN_CAP) r.patch = 2;             // crowded tile: the consumers scan the lists
            return r;
        };
        const unsigned long long l2_policy = l2_evict_first_policy();
        // Work queue: one counter of items.  A CTA first asks for `chunk` consecutive items (seven eighths of an
        // even share: a contiguous run like a static split would give it) and then for single items, each
        // requested one tile ahead (lane 0 keeps the raw result of the atomic until it is needed, so nothing
        // waits for it).  The single items even out the tail and whatever CTAs that started late did not take.
        unsigned int *queue = P.error + WS_QUEUE;
        int run_lo = nitems, run_hi = nitems, nxt_raw = nitems;
        if (lane == 0) run_lo = (int)atomicAdd(queue, (unsigned int)chunk);
        run_lo = __shfl_sync(0xFFFFFFFFu, run_lo, 0);
        run_hi = min(run_lo + chunk, nitems);
        if (lane == 0 && run_lo < nitems) nxt_raw = (int)atomicAdd(queue, 1u);
        auto current_item = [&]() -> int { return run_lo < run_hi ? run_lo : -1; };
        auto advance = [&]() {
            ++run_lo;
            if (run_lo >= run_hi) {
                run_lo = __shfl_sync(0xFFFFFFFFu, nxt_raw, 0);
                run_hi = min(run_lo + 1, nitems);
                if (lane == 0 && run_lo < nitems) nxt_raw = (int)atomicAdd(queue, 1u);
            }
        };
        int n = 0;
        Prep p_next{0, 0, 0};
        int item = current_item();
        bool prepared = false;
        // lane 0: the tile's bulk copy, with the arrival on full[s] (arrive == true) or with the bytes announced only
        // (the arrival then follows once the stage's description is written)
        auto issue_copy = [&](int row, int tile, int s, bool arrive) {
            const int first = tile * CTA_TILE;
            const int elems = min(CTA_TILE, ((P.V - first) + VEC - 1) / VEC * VEC);
            const unsigned int bytes = (unsigned int)elems * ELT;
            const unsigned char *src = reinterpret_cast<const unsigned char *>(P.logits) +
                                       ((size_t)row * (size_t)P.row_stride + (size_t)first) * ELT;
            if (arrive) mbar_arrive_expect_tx(&sh.full[s], bytes); else mbar_expect_tx(&sh.full[s], bytes);
#ifdef SONIC_TEST_WITHHOLD
            // test-only build: the bytes of one chosen tile are announced but its copy is never issued, so the waits
            // on this stage run out (consumers, then the producer) and the call reports it
            if (__ldcg(&P.error[WS_TEST_WITHHOLD]) == (unsigned int)(row * tiles + tile) + 1u) return;
#endif
            bulk_load(stages + (size_t)s * STAGE_BYTES, src, bytes, &sh.full[s], l2_policy);
        };
        // The CTA's first tile is requested at once, before its row's parameters and lists are known (they take two
        // rounds of global loads): the copy's latency hides behind them.  (A row of the cluster kernel's class gets
        // a copy nobody reads: such rows are rare.)
        if (item >= 0 && lane == 0) issue_copy(item / tiles, item % tiles, 0, false);
        for (;; ++n) {
            const int s = n % NSTAGE;
            if (n >= NSTAGE) {
                // the consumers have left tile n - NSTAGE: its stage and its hit buffer are free
                if (!mbar_wait(&sh.empty[s], ((n / NSTAGE) - 1) & 1)) {
                    if (lane == 0) atomicOr(P.error, ERR_TIMEOUT);
                    return;
                }
            }
            if (item < 0) {                            // out of work: tell the consumers
                if (lane == 0) { sh.meta[s].stop = 1; mbar_arrive(&sh.full[s]); }
                break;
            }
            const int row = item / tiles, tile = item - row * tiles;
            if (!prepared) {                           // the CTA's first tile: nothing was prepared ahead
                p_next = prepare(row, tile, n % (NSTAGE + 1));
                prepared = true;
            }
            const RowCfg c = c_next;
            const Prep pr = p_next;
            const int bad_now = row_bad;
            advance();
            const int nxt = current_item();
            __syncwarp();                              // the hit buffer's entries, written by all lanes, precede the arrival
            if (lane == 0) {
                StageMeta &m = sh.meta[s];
                m.cfg = c; m.row = row; m.tile = tile; m.skip = (c.cls == CLS_EXACT) ? 1 : 0;
                m.patch = pr.patch; m.npen = pr.npen; m.nbias = pr.nbias; m.hb = n % (NSTAGE + 1);
                m.stop = 0;
                m.bad = bad_now;
                m.next_row = (nxt >= 0) ? nxt / tiles : -1;
                m.next_tile = (nxt >= 0) ? nxt % tiles : -1;
                if (n == 0 || c.cls == CLS_EXACT) mbar_arrive(&sh.full[s]);     // (the first tile's copy is under way; nothing is copied for rows of the cluster kernel's class)
                else issue_copy(row, tile, s, true);
            }
            __syncwarp();
            // hit buffer (n + 1) % (NSTAGE + 1) was last used by tile n - NSTAGE, which the consumers have left
            if (nxt >= 0) p_next = prepare(nxt / tiles, nxt % tiles, (n + 1) % (NSTAGE + 1));
            item = nxt;
        }
        return;
    }

    // ---------------------------------------------------------------- consumer warps
    // The grammar words of a warp tile (32 words, one coalesced load, handed to the lanes that need them by
    // shuffles later) are requested one tile ahead: each stage names the tile that follows it.
    uint32_t mword_pre = 0u;
    int pre_row = -1, pre_tile = -1;
    auto load_mask_words = [&](int row, int tile) -> uint32_t {
        const int w = ((tile * CTA_TILE + warp * WARP_TILE) >> 5) + lane;
        return (w < ((P.V + 31) >> 5)) ? __ldg(P.bitmask + (size_t)row * P.bitmask_stride + w) : 0u;
    };
    for (int n = 0;; ++n) {
        const int s = n % NSTAGE;
        if (!mbar_wait(&sh.full[s], (n / NSTAGE) & 1)) {
            if (lane == 0) atomicOr(P.error, ERR_TIMEOUT);
            return;
        }
        if (sh.meta[s].stop) { KERNEL_T1(0); break; }
        const int row = sh.meta[s].row, tile = sh.meta[s].tile;
        const int tile_base = tile * CTA_TILE;
        const int wbase = tile_base + warp * WARP_TILE;
        uint32_t mword = 0xFFFFFFFFu;
        if (P.bitmask) {
            mword = (row == pre_row && tile == pre_tile) ? mword_pre : load_mask_words(row, tile);
            pre_row = sh.meta[s].next_row; pre_tile = sh.meta[s].next_tile;
            if (pre_row >= 0) mword_pre = load_mask_words(pre_row, pre_tile);
        }
        const StageMeta &meta = sh.meta[s];
        if (meta.skip) {
            // a row of the cluster kernel: counted, its status word initialised
            if (tile == 0 && tid == 0) { P.rs[row].status = 0u; atomicAdd(&P.error[WS_NEXACT], 1u); }
        } else {
            const RowCfg c = meta.cfg;
            RowState *rs = P.rs + row;
            TileRec *rec = P.tiles + (size_t)row * MAX_TILES + tile;
            // Every per-row word of the workspace is initialised by the call that reads it: the tile's flags here
            // (before any barrier of this tile), the row's status word and, for rows of the histogram path, the
            // row's control block and its histogram by the CTA of the row's first tile.
            if (tid == 0) {
                rec->flags = meta.bad ? TILE_BADID : 0u;
                if (tile == 0) rs->status = 0u;
            }
            if (c.cls == CLS_DENSE && tile == 0) {
                uint4 *h = reinterpret_cast<uint4 *>(P.hist + (size_t)row * DBINS);
                for (int i = tid; i < DBINS / 2; i += STREAM_THREADS) h[i] = make_uint4(0u, 0u, 0u, 0u);
                if (tid == 0) {
                    DenseRow *dr = P.drow + row;
                    dr->ticket_h = 0u; dr->ticket_c = 0u; dr->ticket_r = 0u; dr->nmembers = 0u;
                    dr->kmin = 0xFFFFFFFFu; dr->kmax = 0u; dr->overflow = 0u; dr->state = 0u;
                    P.dlist[atomicAdd(&P.error[WS_NDENSE], 1u)] = row;
                }
            }
            unsigned char *stage = stages + (size_t)s * STAGE_BYTES;
            const bool masked = (c.z & M_GRAMMAR) != 0;
            const bool tail = tile_base + CTA_TILE > P.V;
            const int patch = meta.patch;
            const bool patched = patch != 0;
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
            auto widen = [&]() {                      // bf16 only: the warp's part of the tile as fp32 in shared memory
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    float *p = conv + warp * WARP_TILE + j * 32 * VEC + lane * VEC;
#pragma unroll
                    for (int q = 0; q < VEC; q += 4)
                        *reinterpret_cast<float4 *>(p + q) = make_float4(e[j * VEC + q], e[j * VEC + q + 1], e[j * VEC + q + 2], e[j * VEC + q + 3]);
                }
            };
            // penalties and biases commute with the mask (a masked logit stays -inf), so they are applied to
            // the unmasked tile and the mask is applied when the lanes read their elements
            if (patch == 1) {
                // the producer listed this tile's entries: every warp patches its own part, no block-wide barrier
                if (DT == 1) { read_raw(); widen(); }
                __syncwarp();
                for (int h = lane; h < meta.npen; h += 32) {
                    const Hit x = sh.pen[meta.hb][h];
                    if (x.li / WARP_TILE == warp) ptile[x.li] = apply_penalties(ptile[x.li], x.payload, c);
                }
                __syncwarp();
                for (int h = lane; h < meta.nbias; h += 32) {
                    const Hit x = sh.bias[meta.hb][h];
                    if (x.li / WARP_TILE == warp) ptile[x.li] = __fadd_rn(ptile[x.li], __int_as_float(x.payload));
                }
                __syncwarp();
                read_f32(ptile);
            } else if (patch == 2) {
                // long or crowded lists: all consumer threads scan them together
                if (DT == 1) { read_raw(); widen(); csync(); }
                const int req = (P.op == OP_VERIFY) ? row / (P.K + 1) : row;
                const int *hid = P.hist_ids + (size_t)req * P.hist_stride;
                const int *hct = P.hist_counts + (size_t)req * P.hist_stride;
                bool bad = false;
                for (int t = tid; t < c.hist_len; t += STREAM_THREADS) {
                    const int id = __ldg(hid + t);
                    if (id < 0 || id >= P.V) { bad = true; continue; }
                    const int li = id - tile_base;
                    if (li >= 0 && li < CTA_TILE) ptile[li] = apply_penalties(ptile[li], __ldg(hct + t), c);
                }
                csync();
                for (int t = tid; t < c.bias_len; t += STREAM_THREADS) {
                    const int id = __ldg(P.bias_ids + (size_t)req * P.bias_stride + t);
                    if (id < 0 || id >= P.V) { bad = true; continue; }
                    const int li = id - tile_base;
                    if (li >= 0 && li < CTA_TILE) ptile[li] = __fadd_rn(ptile[li], __ldg(P.bias_vals + (size_t)req * P.bias_stride + t));
                }
                if (bad) atomicOr(&rec->flags, TILE_BADID);          // (ordered after the first thread's store by the barriers above)
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
                for (int q = 0; q < EPL; ++q) e[q] = div_tau(e[q], c.tau);
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
            float qm[4];                               // maxima of the lane's four quarters (8 elements each)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                qm[i] = mv[i * (NV / 4)];
#pragma unroll
                for (int j = 1; j < NV / 4; ++j) qm[i] = fmaxf(qm[i], mv[i * (NV / 4) + j]);
            }
            const float h0 = fmaxf(qm[0], qm[1]), h1 = fmaxf(qm[2], qm[3]);
            const float lm = fmaxf(h0, h1);

            if (c.cls == CLS_GREEDY || c.cls == CLS_DENSE) {
                if (c.cls == CLS_DENSE) {
                    // histogram path: the processed logits (already divided by the temperature) are kept as ordered
                    // keys for the later passes; per tile the smallest finite key and the number of finite elements
                    uint32_t kmn = 0xFFFFFFFFu;
                    unsigned int nf = 0u;
                    unsigned int *yk = P.ykeys + (size_t)row * ((size_t)P.ytiles * CTA_TILE) + tile_base + warp * WARP_TILE;
#pragma unroll
                    for (int j = 0; j < NV; ++j) {
#pragma unroll
                        for (int q4 = 0; q4 < VEC; q4 += 4) {
                            uint32_t kk[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                kk[u] = okey(e[j * VEC + q4 + u]);
                                const bool fin = kk[u] > KEY_NEG_INF;
                                nf += fin ? 1u : 0u;
                                kmn = fin ? min(kmn, kk[u]) : kmn;
                            }
                            *reinterpret_cast<uint4 *>(yk + j * 32 * VEC + lane * VEC + q4) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
                        }
                    }
                    kmn = __reduce_min_sync(0xFFFFFFFFu, kmn);
                    nf = __reduce_add_sync(0xFFFFFFFFu, nf);
                    if (lane == 0) { sh.kmin[s][warp] = kmn; sh.nfin[s][warp] = nf; }
                }
                float wm = lm;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xFFFFFFFFu, wm, off));
                unsigned long long key = 0ull;
                if (wm > -CUDART_INF_F) {
                    int best = 0x7FFFFFFF;
                    if (lm == wm) {
                        // slots ascend: the last write is the lowest; only the first quarter that holds the maximum is searched
                        bool found = false;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (!found && qm[i] == wm) {
                                found = true;
#pragma unroll
                                for (int q = (i + 1) * (EPL / 4) - 1; q >= i * (EPL / 4); --q)
                                    if (e[q] == wm) best = slot_index<DT>(wbase, lane, q);
                            }
                        }
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
                    if (c.cls == CLS_DENSE) {
                        unsigned int kmn = sh.kmin[s][0], nf = sh.nfin[s][0];
#pragma unroll
                        for (int w = 1; w < STREAM_WARPS; ++w) { kmn = min(kmn, sh.kmin[s][w]); nf += sh.nfin[s][w]; }
                        rec->minkey = kmn; rec->nfin = nf;
                    }
                }
            } else {
                // warp cutoff: minimum over G groups of the group maximum.  Tile cutoff: the largest of the eight
                // warp cutoffs (warp mode) or the smallest (tile mode: a minimum over all 8 G groups of the tile).
                // In tile mode a group without a finite element (masked, or past the row's end) does not take
                // part: it would drag the cutoff to -inf and the tile would emit everything it has.
                float g;
                const int G = c.G;
                const bool tmin = c.tile_min;
                switch (G) {                                   // (one straight-line butterfly per group count)
                case 0: g = -CUDART_INF_F; break;
                case 1: g = warp_cutoff<32>(lm, tmin); break;
                case 2: g = warp_cutoff<16>(lm, tmin); break;
                case 4: g = warp_cutoff<8>(lm, tmin); break;
                case 8: g = warp_cutoff<4>(lm, tmin); break;
                case 16: g = warp_cutoff<2>(lm, tmin); break;
                case 32: g = warp_cutoff<1>(lm, tmin); break;
                default: {                                     // 64: half-lane groups
                    const float a0 = (tmin && h0 == -CUDART_INF_F) ? CUDART_INF_F : h0;
                    const float a1 = (tmin && h1 == -CUDART_INF_F) ? CUDART_INF_F : h1;
                    g = warp_cutoff<1>(fminf(a0, a1), false);
                    break;
                }
                }
                if (lane == 0) sh.tw[s][warp] = g;
                if (tid == 0) { sh.ncand[s] = 0; rec->cnt = 0u; }          // (the warps add to the record after the barrier)
                csync();
                static_assert(STREAM_WARPS == 8, "the eight warp cutoffs are read as two 128-bit words");
                const float4 ta = *reinterpret_cast<const float4 *>(&sh.tw[s][0]);
                const float4 tb = *reinterpret_cast<const float4 *>(&sh.tw[s][4]);
                float t;
                if (tmin) {
                    t = fminf(fminf(fminf(ta.x, ta.y), fminf(ta.z, ta.w)), fminf(fminf(tb.x, tb.y), fminf(tb.z, tb.w)));
                    if (t == CUDART_INF_F) t = -CUDART_INF_F;          // no finite element in the tile: nothing to emit
                } else {
                    t = fmaxf(fmaxf(fmaxf(ta.x, ta.y), fmaxf(ta.z, ta.w)), fmaxf(fmaxf(tb.x, tb.y), fmaxf(tb.z, tb.w)));
                }
                // every finite element >= t goes to the tile's candidate slot; a warp reserves its share of the
                // slot with one shared-memory atomic and adds it to the tile record (no second barrier).
                // Most warps hold no candidate at all and leave after one vote.  The others mark their
                // candidates in a bit mask and fetch the values again from the tile in shared memory (a
                // candidate is neither masked nor past the row's end, so the tile holds its value).
                const float t2 = fmaxf(t, -CUDART_MAX_NORMAL_F);           // e >= t2  <=>  e >= t and e is not -inf
                if (__any_sync(0xFFFFFFFFu, lm >= t2)) {
                    // a quarter of the lanes' elements without a candidate anywhere in the warp is skipped by one vote
                    unsigned int cm = 0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (__any_sync(0xFFFFFFFFu, qm[i] >= t2)) {
#pragma unroll
                            for (int q = i * (EPL / 4); q < (i + 1) * (EPL / 4); ++q) cm |= (e[q] >= t2) ? (1u << q) : 0u;
                        }
                    }
                    const int cnt = __popc(cm);
                    int incl, total;
                    if (!__any_sync(0xFFFFFFFFu, cnt > 1)) {
                        // the usual case, at most one candidate per lane: positions from one vote
                        const unsigned int has = __ballot_sync(0xFFFFFFFFu, cnt > 0);
                        incl = __popc(has & (0xFFFFFFFFu >> (31 - lane)));
                        total = __popc(has);
                    } else {
                        incl = cnt;
#pragma unroll
                        for (int off = 1; off < 32; off <<= 1) {
                            const int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                            if (lane >= off) incl += o;
                        }
                        total = __shfl_sync(0xFFFFFFFFu, incl, 31);
                    }
                    unsigned int base = 0;
                    if (lane == 0) {
                        base = atomicAdd(&sh.ncand[s], (unsigned int)total);
                        atomicAdd(&rec->cnt, (unsigned int)total);      // zero before the call; the merge kernel clears it
                    }
                    base = __shfl_sync(0xFFFFFFFFu, base, 0);
                    if ((int)base + total <= cap_t) {
                        unsigned long long *dst = P.cand + (size_t)row * P.cand_stride + (size_t)tile * cap_t + base + (incl - cnt);
                        const int lbase = warp * WARP_TILE + lane * VEC;
                        while (cm) {
                            const int q = __ffs(cm) - 1;
                            cm &= cm - 1;
                            const int li = lbase + (q / VEC) * (32 * VEC) + (q % VEC);
                            float v;
                            if (DT == 0 || patched) v = ptile[li];
                            else v = __uint_as_float((uint32_t)reinterpret_cast<const unsigned short *>(stage)[li] << 16);
                            if (c.div_all) v = div_tau(v, c.tau);
                            *dst++ = ((unsigned long long)okey(v) << 32) | (uint32_t)(~(uint32_t)(tile_base + li));
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
// cluster kernel.
__global__ void __launch_bounds__(MERGE_THREADS, 2)
sonic_merge_kernel(const KParams P, const int tiles) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ MergeShared<MERGE_THREADS> s_merge;
    const int row = blockIdx.x;
    const int tid = threadIdx.x;
    KERNEL_T0(1);
    const RowCfg c = load_cfg(P, row);         // inputs only: independent of the streaming kernel
    const bool other = (c.cls == CLS_EXACT || c.cls == CLS_DENSE);
    if (other && row != 0) return;
    // the row's two uniforms depend on the inputs alone: drawn here, while the streaming kernel may still be running
    uint2 cells = make_uint2(0u, 0u);
    if (P.op != OP_TOPK && c.cls == CLS_TOPK) draw_cells(P, c, cells.x, cells.y);
    pdl_wait_primary();                        // tile records and candidates of the streaming kernel
    // The next kernel of the call (stage 2 of the histogram path) does not wait for this grid: it needs the
    // streaming kernel's results only, and those are complete once every CTA here is past its wait (the first
    // row's CTA never leaves before it).  So it is let go after the wait, and runs beside the merges.
    pdl_launch_dependents();
    if (row == 0 && tid == 0) P.error[WS_QUEUE] = 0u;    // the streaming kernel is done with its work counter
    if (other) return;
    if (__ldcg(&P.error[WS_ERROR]) & ERR_TIMEOUT) {
        // a bounded wait of the streaming kernel ran out (in this call or an earlier one on this workspace): the
        // tile records are not to be trusted, the row reports it instead of a token
        if (tid == 0) {
            if (P.op == OP_TOPK) { for (int j = 0; j < P.ktop; ++j) { P.out_vals[(size_t)row * P.ktop + j] = -CUDART_INF_F; P.out_idx[(size_t)row * P.ktop + j] = -1; } }
            else emit_row(P, c, row, -1, 0.0f, F_TIMEOUT, 0, 0.0f);
        }
        return;
    }
    RowState *rs = P.rs + row;
    const TileRec *recs = P.tiles + (size_t)row * MAX_TILES;
    const unsigned int tflags = (tid < tiles) ? __ldcg(&recs[tid].flags) : 0u;
    const bool badid = __syncthreads_or((int)(tflags & TILE_BADID)) != 0;
    if (c.bad || badid) {
        if (tid == 0) emit_row(P, c, row, -1, 0.0f, F_BADPARAM, 0, 0.0f);
        return;
    }
    if (c.cls == CLS_GREEDY) {
        if (tid < 32) {
            unsigned long long best = (tid < tiles) ? __ldcg(&recs[tid].best) : 0ull;
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
    const bool ok = merge_topk_row<MERGE_THREADS, BlockSync>(P, c, row, tiles, reinterpret_cast<unsigned long long *>(smem_raw), s_merge, tid, cells);
    if (tid == 0 && !ok) { rs->status = ST_FAILED; atomicAdd(&P.error[WS_FAILED_ROWS], 1u); }
    KERNEL_T1(1);
}

}  // namespace sonic
