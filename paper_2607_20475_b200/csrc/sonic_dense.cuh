// Histogram path: rows with top-k off (top-p, min-p or plain temperature sampling over the whole vocabulary,
// and their verification variants), finished by grid-wide passes over the row's ordered keys instead of by one
// cluster per row.
//
// The streaming kernel leaves, per row of this class, the ordered keys of the processed logits (read once from
// HBM, written once, re-read from L2 by the passes below) and per-tile maxima / minima.  Then, every pass a
// grid-wide launch whose CTAs take (row, tile) items and whose last-arriving CTA of a row (a ticket counter, no
// waiting) does the row-level step:
//   pass H  (rows with top-p): fixed-point probability mass per bin, 2048 bins uniform in (M - y) that just cover
//           the row's finite range; the last arriver scans the bins from the top for the bin where the
//           cumulative mass reaches p * Z (the "crossing bin").  The min-p threshold M + ln(theta) is a key
//           threshold and names a bin as well; the higher of the two bins decides.
//   pass C  per tile: mass and number of the elements above the crossing bin, and the elements inside it listed
//           as (key << 32 | ~index); the last arriver resolves the exact cut among the listed elements (a radix
//           descent over the composite keys weighted by mass; ties by lowest index), then draws: tile-level
//           CDF from the per-tile masses, one tile re-read for the element.  Rows without top-p know their cut
//           once the row maximum is known and run pass C in place of pass H.
//   pass R  (verification rows whose draft was rejected): per-tile sums of the residual max(0, p - q) in fp64,
//           the last arriver draws from it.
// This is the truncation epilogue and token selection of the paper's Algorithm "Stage 2" (TopP, MinP; Appendix
// "Probability Truncation", "Sampling", "Speculative Verification") for supports far beyond the paper's
// k <= 128 bound (Section 3.3).  Masses are 2^-40 fixed point, sums are integer and order-independent.
#pragma once
#include "sonic_common.cuh"

namespace sonic {


constexpr int DENSE_THREADS = 512;
constexpr int DENSE_WARPS = DENSE_THREADS / 32;
constexpr int DENSE_EPT = CTA_TILE / DENSE_THREADS;          // 16 keys per thread and tile
constexpr int DENSE_NV = DENSE_EPT / 4;                      // as 128-bit vectors
constexpr int STAGE_CAP = 2048;                              // elements of the crossing bin one item can stage
constexpr int DENSE_DYN_SMEM = MEMBER_CAP * 8;               // members | histogram words | staged members share it
static_assert(DBINS * 8 <= DENSE_DYN_SMEM && STAGE_CAP * 8 <= DENSE_DYN_SMEM, "dynamic shared memory of the dense passes");
static_assert(MAX_TILES == 32, "one tile record per lane");
static_assert(MAX_TILES * DENSE_CHUNKS == DENSE_THREADS, "one chunk record per thread");

struct DenseShared {
    unsigned long long tile_mass[MAX_TILES];
    unsigned int tile_nb[MAX_TILES];
    unsigned long long red64[DENSE_WARPS];
    double redd[3][DENSE_WARPS];
    unsigned int red32[2][DENSE_WARPS];
    unsigned long long comp[DENSE_THREADS];          // listed elements (fast path: at most one per thread)
    unsigned long long wt[DENSE_THREADS];            // their weights in ranking order
    unsigned long long chunk[DENSE_THREADS];         // support mass per chunk of 512 elements (tile-major)
    unsigned int sub[5][DENSE_THREADS];              // medium path of the finish: per sub-bin count, mass words, smallest and largest key
    unsigned long long bc64[4];
    double bcd[2];
    unsigned int nstage, kmin, kmax, base;
    unsigned int Mkey, mkey, Nf, bad;
    unsigned int cnt_above, nb;
    int flag, last, digit;
};

// Bin of a finite key: larger bin = larger logit; bin DBINS-1 holds the row maximum.
__device__ __forceinline__ int dense_digit(uint32_t key, float Mf, float scale) {
    const float t = fminf(__fmul_rn(__fsub_rn(Mf, unkey(key)), scale), (float)(DBINS - 1));
    return DBINS - 1 - (int)t;
}

// Bins per logit unit, a power of two chosen so that the bins just cover the row's finite range.
__device__ __forceinline__ float dense_scale(uint32_t Mkey, uint32_t mkey, unsigned int Nf) {
    int e = 5;
    const float spread = (Nf > 0) ? __fsub_rn(unkey(Mkey), unkey(mkey)) : 0.0f;
    if (spread > 0.0f && spread < CUDART_INF_F) e = max(-10, min(10, ilogbf((float)(DBINS - 8) / spread)));
    return ldexpf(1.0f, e);
}

// Smallest key in (okey(-inf), Mkey] whose bin is at least b (Mkey + 1 if none): the bins are monotone in the
// key, so a 32-way search by one warp finds it in seven rounds.  Every lane returns the result.
__device__ __forceinline__ uint32_t dense_bin_lower_key(int b, uint32_t Mkey, float Mf, float scale, int lane) {
    uint32_t lo = KEY_NEG_INF + 1u, hi = Mkey + 1u;           // the answer lies in [lo, hi]
    while (lo < hi) {
        const uint32_t step = (hi - lo) / 32u + 1u;
        const unsigned long long cand64 = (unsigned long long)lo + (unsigned long long)lane * step;
        const bool valid = cand64 < (unsigned long long)hi;
        const uint32_t cand = (uint32_t)cand64;
        const bool ok = valid && dense_digit(cand, Mf, scale) >= b;
        const unsigned int m = __ballot_sync(0xFFFFFFFFu, ok);
        const unsigned int v = __ballot_sync(0xFFFFFFFFu, valid);
        if (m == 0u) {
            lo = lo + (uint32_t)(31 - __clz(v)) * step + 1u;     // past the last candidate (lane 0's is always valid)
        } else {
            const int l = __ffs(m) - 1;
            hi = lo + (uint32_t)l * step;
            if (l > 0) lo = lo + (uint32_t)(l - 1) * step + 1u; else hi = lo;
        }
    }
    return lo;
}

__device__ __forceinline__ unsigned long long dense_warp_sum(unsigned long long v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

// Inclusive scan over the lanes of a warp.
__device__ __forceinline__ unsigned long long dense_warp_scan(unsigned long long v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, v, o);
        if (lane >= o) v += up;
    }
    return v;
}

// Exclusive prefix over the threads of the block (thread order) of one value per thread; `total` in every thread.
template <typename T>
__device__ __forceinline__ T dense_block_scan(T v, T *wtot, int tid, T &total) {
    const int lane = tid & 31, warp = tid >> 5;
    T incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += up;
    }
    __syncthreads();
    if (lane == 31) wtot[warp] = incl;
    __syncthreads();
    T off = T(0), tot = T(0);
#pragma unroll
    for (int w = 0; w < DENSE_WARPS; ++w) {
        const T t = wtot[w];
        if (w < warp) off += t;
        tot += t;
    }
    total = tot;
    return off + incl - v;
}

// Row statistics from the streaming kernel's tile records (first warp): maximum, smallest finite key, finite count.
__device__ __forceinline__ void dense_row_stats(const KParams &P, int row, int tiles, DenseShared &sm, int tid) {
    if (tid < 32) {
        const TileRec *rec = P.tiles + (size_t)row * MAX_TILES;
        unsigned int mk = 0u, mn = 0xFFFFFFFFu, nf = 0u, fl = 0u;
        if (tid < tiles) {
            mk = (unsigned int)(rec[tid].best >> 32);
            mn = rec[tid].minkey;
            nf = rec[tid].nfin;
            fl = rec[tid].flags;
        }
        mk = __reduce_max_sync(0xFFFFFFFFu, mk);
        mn = __reduce_min_sync(0xFFFFFFFFu, mn);
        nf = __reduce_add_sync(0xFFFFFFFFu, nf);
        fl = __reduce_or_sync(0xFFFFFFFFu, fl);
        if (tid == 0) { sm.Mkey = mk; sm.mkey = mn; sm.Nf = nf; sm.bad = fl & TILE_BADID; }
    }
}

// Work items of a pass: a tile is cut into `sub` parts (1, 2 or 4) when the call has so few rows of this class that
// whole tiles would leave most SMs idle.  A thread holds 16 / sub consecutive elements of its part, so a chunk of
// 512 elements belongs to `sub` consecutive warps.
struct DenseItem {
    int row, tile, part, sub;
    __device__ int nv() const { return DENSE_NV / sub; }                       // 128-bit vectors per thread
    __device__ int first(int tid) const { return tile * CTA_TILE + part * (CTA_TILE / sub) + tid * (DENSE_EPT / sub); }
};
__device__ __forceinline__ int dense_pick_sub(int rows_in_pass, int tiles, int ctas) {
    int sub = 1;
    while (sub < 4 && rows_in_pass * tiles * sub * 2 <= ctas) sub *= 2;
    return sub;
}
// `head`: the lane's entry of the list's first 32 (requested together with the list's length, so that a CTA's first row
// is known after one round trip instead of two); every thread of the CTA calls this at the same point.
__device__ __forceinline__ DenseItem dense_item(const int *list, int head, int item, int tiles, int sub) {
    DenseItem it;
    const int per_row = tiles * sub;
    const int slot = item / per_row;
    const int from_head = __shfl_sync(0xFFFFFFFFu, head, slot & 31);
    it.row = (slot < 32) ? from_head : __ldcg(&list[slot]);
    const int rem = item % per_row;
    it.tile = rem / sub; it.part = rem % sub; it.sub = sub;
    return it;
}

// The item's keys.  They were written by an earlier kernel of the call, so the loads may go through L1 (the loads
// of a thread share their lines).  Vectors past the item's share hold okey(-inf).
__device__ __forceinline__ void dense_load_keys(const KParams &P, const DenseItem &it, int tid, uint4 (&kv)[DENSE_NV]) {
    const uint4 *src = reinterpret_cast<const uint4 *>(P.ykeys + (size_t)it.row * ((size_t)P.ytiles * CTA_TILE) + it.first(tid));
    const int nv = it.nv();
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) kv[k] = (k < nv) ? src[k] : make_uint4(KEY_NEG_INF, KEY_NEG_INF, KEY_NEG_INF, KEY_NEG_INF);
}

// Ticket of a pass: a CTA reports `cnt` finished items of a row at once; true in every thread of the CTA whose report
// completes the row's `items` (its reads then see what the others wrote).
__device__ __forceinline__ bool dense_arrive(unsigned int *ticket, int cnt, int items, DenseShared &sm, int tid) {
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(ticket, (unsigned int)cnt);
        sm.last = (t + (unsigned int)cnt == (unsigned int)items) ? 1 : 0;
        if (sm.last) __threadfence();
    }
    __syncthreads();
    return sm.last != 0;
}

// The items of a pass are dealt in contiguous ranges, so that a CTA's items mostly belong to one row: the row's
// parameters are loaded once, its ticket is drawn once, and the rows a CTA turns out to complete are finished after
// all of its items (another row's items never wait behind a finish).
struct DenseRange { int lo, hi; };
__device__ __forceinline__ DenseRange dense_range(int n_items, int cta, int ncta) {
    const int per = (n_items + ncta - 1) / ncta;
    DenseRange r;
    r.lo = min(n_items, cta * per);
    r.hi = min(n_items, r.lo + per);
    return r;
}
constexpr int DENSE_FIN_MAX = 8;              // rows one CTA can have to finish (a range spans few rows)

// ---------------------------------------------------------------- pass H
// Mass histogram of one item, added to the row's histogram in global memory.
__device__ __forceinline__ void dense_hist_item(const KParams &P, const DenseItem &it, const uint4 (&kv)[DENSE_NV], float Mf, float scale,
                                                unsigned int *hm0, unsigned int *hm1, int tid) {
    for (int i = tid; i < DBINS; i += DENSE_THREADS) { hm0[i] = 0u; hm1[i] = 0u; }
    __syncthreads();
    const int nv = it.nv();
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) {
        if (k >= nv) break;
        const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
        int bin[4];
        unsigned long long q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const bool fin = key4[u] > KEY_NEG_INF;
            const int dg = dense_digit(key4[u], Mf, scale);
            const unsigned long long wq = qweight(key4[u], Mf);
            bin[u] = fin ? dg : -1;
            q[u] = fin ? wq : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (bin[u] < 0 || q[u] == 0ull) continue;
            // 64-bit mass as two 32-bit words: the low word's returned old value reveals a carry
            const unsigned int lo = (unsigned int)q[u], hi = (unsigned int)(q[u] >> 32);
            unsigned int carry = 0;
            if (lo) { const unsigned int old = atomicAdd(&hm0[bin[u]], lo); carry = (old + lo < old) ? 1u : 0u; }
            if (hi + carry) atomicAdd(&hm1[bin[u]], hi + carry);
        }
    }
    __syncthreads();
    unsigned long long *hist = P.hist + (size_t)it.row * DBINS;
    for (int i = tid; i < DBINS; i += DENSE_THREADS) {
        const unsigned long long m = (unsigned long long)hm0[i] | ((unsigned long long)hm1[i] << 32);
        if (m) atomicAdd(&hist[i], m);
    }
}

// Row step of pass H: the crossing bin of top-p against the min-p threshold, as the key interval pass C works with
// (in every thread: klo, khi, tk, target).  Every CTA of pass C that meets the row computes it for itself from the
// row's histogram (16 KB, four bins per thread); `store` (the CTA of the row's first item) leaves it for the row's finish.
struct DenseCut { uint32_t tk, klo, khi; unsigned long long target; };
// A thread's bins of the row's histogram: thread t owns bins DBINS-1-4t .. DBINS-4-4t (from the top).  Requested by the
// caller before the row's other loads are waited for.
constexpr int DENSE_BPT = DBINS / DENSE_THREADS;
struct DenseBins { unsigned long long v[DENSE_BPT]; };
__device__ __forceinline__ DenseBins dense_load_bins(const KParams &P, int row, int tid) {
    const unsigned long long *hist = P.hist + (size_t)row * DBINS;
    DenseBins b;
#pragma unroll
    for (int j = 0; j < DENSE_BPT; ++j) b.v[j] = __ldcg(&hist[DBINS - 1 - (tid * DENSE_BPT + j)]);
    return b;
}
__device__ __forceinline__ DenseCut dense_hist_finish(const KParams &P, const RowCfg &c, int row, DenseShared &sm,
                                                      const DenseBins &bins, int tid, uint32_t Mkey, float scale, bool store) {
    constexpr int BPT = DENSE_BPT;
    unsigned long long mine = 0;
#pragma unroll
    for (int j = 0; j < BPT; ++j) mine += bins.v[j];
    unsigned long long Z;
    const unsigned long long pre = dense_block_scan<unsigned long long>(mine, sm.red64, tid, Z);
    unsigned long long target = (unsigned long long)ceil((double)c.p * (double)Z);
    if (target > Z) target = Z;
    if (target < 1ull) target = 1ull;
    if (tid == 0) sm.digit = 0;
    __syncthreads();
    if (mine > 0ull && pre < target && target <= pre + mine) {
        unsigned long long cum = pre;
        int found = -1;
#pragma unroll
        for (int j = 0; j < BPT; ++j) {
            const int b = DBINS - 1 - (tid * BPT + j);
            cum += bins.v[j];
            if (found < 0 && cum >= target) found = b;
        }
        sm.digit = found;
    }
    __syncthreads();
    if (tid < 64) {
        // two warps: the lower key of the bin, and the lower key of the bin above it
        const float Mf = unkey(Mkey);
        const int b_p = sm.digit;
        uint32_t tk = 0u;
        int b_m = -1;
        if (c.z & M_MIN_P) { tk = minp_key(Mf, c.theta); b_m = dense_digit(max(tk, KEY_NEG_INF + 1u), Mf, scale); }
        if (b_m > b_p) {
            // the min-p threshold lies above the bin top-p would cut in: the cut is the threshold itself
            if (tid == 0) { sm.bc64[0] = ((unsigned long long)0xFFFFFFFFu << 32) | (tk - 1u); sm.bc64[1] = 0ull; sm.base = tk; }
        } else {
            const uint32_t k = dense_bin_lower_key(b_p + (tid >> 5), Mkey, Mf, scale, tid & 31);
            if (tid == 32) sm.kmax = k - 1u;                    // khi
            if (tid == 0) { sm.kmin = k; sm.bc64[1] = target; sm.base = tk; }     // klo
        }
    }
    __syncthreads();
    DenseCut r;
    if (sm.bc64[1] == 0ull) { r.klo = (uint32_t)(sm.bc64[0] >> 32); r.khi = (uint32_t)sm.bc64[0]; }
    else { r.klo = sm.kmin; r.khi = sm.kmax; }
    r.tk = sm.base; r.target = sm.bc64[1];
    __syncthreads();
    if (store && tid == 0) {
        DenseRow *dr = P.drow + row;
        dr->Mkey = Mkey; dr->tk = r.tk; dr->klo = r.klo; dr->khi = r.khi; dr->target = r.target;
        dr->state = 1u;
    }
    return r;
}

// ---------------------------------------------------------------- in-tile search
// First element of a tile, in index order, whose inclusive running sum of wf exceeds `rest`; thread t owns the
// 16 consecutive elements 16t .. 16t + 15.  Returns the element's global index in every thread (the last element
// of positive weight if the sum never exceeds `rest`, -1 if the tile has none) and leaves its weight in w_out.
template <typename T, typename WF>
__device__ int dense_tile_find(const KParams &P, int row, int tile, T rest, WF wf, T *wtot, DenseShared &sm, int tid, T &w_out) {
    const uint4 *src = reinterpret_cast<const uint4 *>(P.ykeys + (size_t)row * ((size_t)P.ytiles * CTA_TILE) + (size_t)tile * CTA_TILE) + tid * DENSE_NV;
    const int first = tile * CTA_TILE + tid * DENSE_EPT;
    uint4 kv[DENSE_NV];
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) kv[k] = src[k];
    if (tid == 0) { sm.flag = -1; sm.digit = -1; }
    T s = T(0);
    int lastpos = -1;
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) {
        const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const T w = wf(key4[u], first + k * 4 + u);
            s += w;
            if (w > T(0)) lastpos = first + k * 4 + u;
        }
    }
    T total;
    const T pre = dense_block_scan<T>(s, wtot, tid, total);
    // weight of the thread's first element whose running sum exceeds `rest` (want_last: of its last positive element)
    auto walk = [&](bool want_last, int &found, T &fw) {
        T cum = pre;
        found = -1; fw = T(0);
#pragma unroll
        for (int k = 0; k < DENSE_NV; ++k) {
            const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const T w = wf(key4[u], first + k * 4 + u);
                cum += w;
                if (w > T(0) && (want_last || (found < 0 && cum > rest))) { found = first + k * 4 + u; fw = w; }
            }
        }
    };
    if (s > T(0) && pre <= rest && rest < pre + s) {
        int found; T fw;
        walk(false, found, fw);
        if (found < 0) walk(true, found, fw);                  // (floating-point sums only)
        sm.flag = found;
        *reinterpret_cast<T *>(&sm.bc64[3]) = fw;
    }
    __syncthreads();
    if (sm.flag < 0) {
        // the running sum never exceeds `rest` (rounding between the levels): the tile's last element of positive weight
        if (lastpos >= 0) atomicMax(&sm.digit, lastpos);
        __syncthreads();
        if (lastpos >= 0 && lastpos == sm.digit) {
            int found; T fw;
            walk(true, found, fw);
            sm.flag = found;
            *reinterpret_cast<T *>(&sm.bc64[3]) = fw;
        }
        __syncthreads();
    }
    w_out = *reinterpret_cast<T *>(&sm.bc64[3]);
    const int res = sm.flag;
    __syncthreads();
    return res;
}

// ---------------------------------------------------------------- pass C
// One item of pass C: per chunk of 512 elements the mass and number of the elements above the crossing bin
// (key > khi) and the number inside it (klo <= key <= khi); the latter staged and appended to the row's member list.
__device__ __forceinline__ void dense_collect_part(const KParams &P, const DenseItem &it, const uint4 (&kv)[DENSE_NV], float Mf,
                                                   uint32_t klo, uint32_t khi, DenseShared &sm, unsigned long long *stage, int tid) {
    const int lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { sm.nstage = 0u; sm.kmin = 0xFFFFFFFFu; sm.kmax = 0u; }
    __syncthreads();
    unsigned long long am = 0ull;
    unsigned int an = 0u, bn = 0u;
    uint32_t kmn = 0xFFFFFFFFu, kmx = 0u;
    const int base_idx = it.first(tid);
    const int nv = it.nv();
    const bool any_members = klo <= khi;
    // the weights first, without a branch per element (the chains of a thread's elements overlap) ...
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) {
        if (k >= nv) break;
        const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned long long w = qweight(key4[u], Mf);
            am += (key4[u] > khi) ? w : 0ull;
            an += (key4[u] > khi) ? 1u : 0u;
        }
    }
    // ... then the elements of the crossing bin, if the row has one
    if (any_members) {
#pragma unroll
        for (int k = 0; k < DENSE_NV; ++k) {
            if (k >= nv) break;
            const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const uint32_t key = key4[u];
                const bool mb = key >= klo && key <= khi;
                const unsigned int mm = __ballot_sync(0xFFFFFFFFu, mb);
                if (mm) {
                    unsigned int pos = 0;
                    if (lane == 0) pos = atomicAdd(&sm.nstage, (unsigned int)__popc(mm));
                    pos = __shfl_sync(0xFFFFFFFFu, pos, 0) + __popc(mm & ((1u << lane) - 1u));
                    if (mb) {
                        if (pos < (unsigned int)STAGE_CAP) stage[pos] = ((unsigned long long)key << 32) | (uint32_t)(~(uint32_t)(base_idx + k * 4 + u));
                        kmn = min(kmn, key); kmx = max(kmx, key);
                        ++bn;
                    }
                }
            }
        }
    }
    am = dense_warp_sum(am);
    an = __reduce_add_sync(0xFFFFFFFFu, an);
    bn = __reduce_add_sync(0xFFFFFFFFu, bn);
    if (any_members) {
        kmn = __reduce_min_sync(0xFFFFFFFFu, kmn);
        kmx = __reduce_max_sync(0xFFFFFFFFu, kmx);
    }
    if (lane == 0) {
        sm.red64[warp] = am; sm.red32[0][warp] = an; sm.red32[1][warp] = bn;
        if (kmx) { atomicMin(&sm.kmin, kmn); atomicMax(&sm.kmax, kmx); }
    }
    __syncthreads();
    // a chunk belongs to `sub` consecutive warps
    const int sub = it.sub, nchunks = DENSE_CHUNKS / sub;
    if (tid < nchunks) {
        DenseChunk r; r.A = 0ull; r.n = 0u; r.nb = 0u;
        for (int w = tid * sub; w < (tid + 1) * sub; ++w) { r.A += sm.red64[w]; r.n += sm.red32[0][w]; r.nb += sm.red32[1][w]; }
        P.dtile[(size_t)it.row * MAX_TILES + it.tile].ch[it.part * nchunks + tid] = r;
    }
    const unsigned int cnt = sm.nstage;
    if (cnt == 0u) return;
    if (tid == 0) {
        DenseRow *dr = P.drow + it.row;
        sm.base = atomicAdd(&dr->nmembers, cnt);
        atomicMin(&dr->kmin, sm.kmin);
        atomicMax(&dr->kmax, sm.kmax);
        if (cnt > (unsigned int)STAGE_CAP) atomicOr(&dr->overflow, 1u);
    }
    __syncthreads();
    const unsigned int base = sm.base;
    unsigned long long *mem = P.members + (size_t)it.row * MEMBER_CAP;
    for (unsigned int i = tid; i < min(cnt, (unsigned int)STAGE_CAP); i += DENSE_THREADS)
        if (base + i < (unsigned int)MEMBER_CAP) mem[base + i] = stage[i];
}

// Sorts the listed elements (composite keys, distinct) in dyn[0, nb) descending, nb > DENSE_THREADS.
__device__ __forceinline__ void dense_sort_members(unsigned long long *dyn, int nb, int tid) {
    const int m = next_pow2(nb);
    for (int i = nb + tid; i < m; i += DENSE_THREADS) dyn[i] = 0ull;
    __syncthreads();
    bitonic_sort_desc_cta<DENSE_THREADS>(dyn, m, tid);
}

// Rank-th (0-based) element of a tile with key == v, in index order.
__device__ __forceinline__ int dense_tile_find_tie(const KParams &P, int row, int tile, uint32_t v, unsigned long long rank,
                                                   DenseShared &sm, int tid) {
    unsigned long long wdummy;
    auto wf = [=](uint32_t key, int) -> unsigned long long { return key == v ? 1ull : 0ull; };
    return dense_tile_find<unsigned long long>(P, row, tile, rank, wf, sm.red64, sm, tid, wdummy);
}

// The draw by one warp, from the support's mass per tile and per chunk (shared memory, final): the tile, then the
// chunk of 512 elements, then the element (a lane owns 16 consecutive elements of the chunk).  Exact: all integer.
// Returns the token in every lane and its weight in qt.
__device__ __forceinline__ int dense_warp_draw(const KParams &P, int row, int tiles, const DenseShared &sm, unsigned long long cutc, float Mf,
                                               unsigned long long T, int lane, unsigned long long &qt) {
    auto pick = [&](unsigned long long v, unsigned long long incl, unsigned long long rest) -> int {
        unsigned int hit = __ballot_sync(0xFFFFFFFFu, v > 0ull && incl > rest);
        if (!hit) { const unsigned int any = __ballot_sync(0xFFFFFFFFu, v > 0ull); hit = any ? (0x80000000u >> __clz(any)) : 1u; }   // (rest < total always: kept for safety)
        return __ffs(hit) - 1;
    };
    // tile
    const unsigned long long tm = (lane < tiles) ? sm.tile_mass[lane] : 0ull;
    const unsigned long long ti = dense_warp_scan(tm, lane);
    const int jt = pick(tm, ti, T);
    const unsigned long long before_t = __shfl_sync(0xFFFFFFFFu, ti - tm, jt);
    unsigned long long rest = (T > before_t) ? T - before_t : 0ull;
    // chunk
    const unsigned long long cm = (lane < DENSE_CHUNKS) ? sm.chunk[jt * DENSE_CHUNKS + lane] : 0ull;
    const unsigned long long ci = dense_warp_scan(cm, lane);
    const int ch = pick(cm, ci, rest);
    const unsigned long long before_c = __shfl_sync(0xFFFFFFFFu, ci - cm, ch);
    rest = (rest > before_c) ? rest - before_c : 0ull;
    // element
    const int first = jt * CTA_TILE + ch * DENSE_CHUNK + lane * 16;
    const uint4 *src = reinterpret_cast<const uint4 *>(P.ykeys + (size_t)row * ((size_t)P.ytiles * CTA_TILE) + first);
    uint4 kv[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) kv[k] = src[k];
    unsigned long long w[16];
    unsigned long long s = 0ull;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = first + k * 4 + u;
            const unsigned long long wq = qweight(key4[u], Mf);
            w[k * 4 + u] = ((((unsigned long long)key4[u] << 32) | (uint32_t)(~(uint32_t)idx)) >= cutc) ? wq : 0ull;
            s += w[k * 4 + u];
        }
    }
    const unsigned long long si = dense_warp_scan(s, lane);
    const int l = pick(s, si, rest);
    int token = -1;
    unsigned long long fw = 0ull;
    if (lane == l) {
        unsigned long long cum = si - s;
        int lastpos = -1;
        unsigned long long lw = 0ull;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            cum += w[i];
            if (w[i] > 0ull) {
                if (token < 0 && cum > rest) { token = first + i; fw = w[i]; }
                lastpos = first + i; lw = w[i];
            }
        }
        if (token < 0) { token = lastpos; fw = lw; }
    }
    token = __shfl_sync(0xFFFFFFFFu, token, l);
    qt = __shfl_sync(0xFFFFFFFFu, fw, l);
    return token;
}

// 64-bit add to a shared-memory word as two native 32-bit atomics (low word first: the value it returns tells whether
// the sum carried).  A 64-bit shared-memory atomic is a compare-and-swap loop, which crawls when many lanes add to a
// handful of words (the per-tile masses of a row: 16 words, hundreds of listed elements).
__device__ __forceinline__ void smem_add_u64(unsigned long long *p, unsigned long long w) {
    unsigned int *q = reinterpret_cast<unsigned int *>(p);
    const unsigned int lo = (unsigned int)w, hi = (unsigned int)(w >> 32);
    unsigned int carry = 0u;
    if (lo) { const unsigned int old = atomicAdd(q, lo); carry = (old + lo < old) ? 1u : 0u; }
    if (hi + carry) atomicAdd(q + 1, hi + carry);
}

// Last arriver of pass C: the exact cut, the support's size and mass, then the draw or the accept test.
// dyn: DENSE_DYN_SMEM bytes; cells: the row's two Philox cells.  Returns false if the row must go to the cluster kernel.
__device__ bool dense_finish(const KParams &P, const RowCfg &c, int row, int tiles, DenseShared &sm, unsigned long long *dyn, int tid,
                             uint32_t Mkey, bool listed, unsigned long long target, uint32_t tk, uint2 cells, int draft, float q_draft) {
    const float Mf = unkey(Mkey);
    const int lane = tid & 31, warp = tid >> 5;
    DenseRow *dr = P.drow + row;
    DenseTile *dt = P.dtile + (size_t)row * MAX_TILES;
    // verification: the draft token's key goes out with the row's other loads (the token itself and its draft
    // probability are inputs, read by the caller before the wait; draft = -1: no draft, or an id outside the vocabulary)
    uint32_t key_draft = 0u;
    if (draft >= 0) key_draft = __ldcg(&P.ykeys[(size_t)row * ((size_t)P.ytiles * CTA_TILE) + draft]);
    // everything the other CTAs left, requested at once: a chunk record per thread, the first DENSE_THREADS listed
    // elements (one per thread, whatever their number turns out to be), their count and the overflow mark
    unsigned int nm = 0u, overflow = 0u;
    {
        const int t = tid / DENSE_CHUNKS;
        DenseChunk r; r.A = 0ull; r.n = 0u; r.nb = 0u;
        if (t < tiles) {
            const uint4 raw = __ldcg(reinterpret_cast<const uint4 *>(&dt[t].ch[tid % DENSE_CHUNKS]));
            r.A = (unsigned long long)raw.x | ((unsigned long long)raw.y << 32); r.n = raw.z; r.nb = raw.w;
        }
        unsigned long long m0 = 0ull;
        if (listed) {
            nm = __ldcg(&dr->nmembers);
            overflow = __ldcg(&dr->overflow);
            m0 = __ldcg(P.members + (size_t)row * MEMBER_CAP + tid);
        }
        sm.chunk[tid] = r.A;
        sm.comp[tid] = ((unsigned int)tid < nm) ? m0 : 0ull;
        // tile sums over 16 consecutive threads, then block sums
        unsigned long long ta = r.A;
        unsigned int tb = r.nb;
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) { ta += __shfl_xor_sync(0xFFFFFFFFu, ta, off); tb += __shfl_xor_sync(0xFFFFFFFFu, tb, off); }
        if ((lane & 15) == 0) { sm.tile_mass[2 * warp + (lane >> 4)] = ta; sm.tile_nb[2 * warp + (lane >> 4)] = tb; }
        const unsigned long long wa = ta + __shfl_xor_sync(0xFFFFFFFFu, ta, 16);
        const unsigned int wn = __reduce_add_sync(0xFFFFFFFFu, r.n);
        if (lane == 0) { sm.red64[warp] = wa; sm.red32[0][warp] = wn; }
        if (tid == 0) { sm.bc64[0] = 0ull; sm.bc64[1] = 0ull; }
    }
    __syncthreads();
    unsigned long long C_above = 0ull;
    unsigned int cnt_above = 0u;
#pragma unroll
    for (int w = 0; w < DENSE_WARPS; ++w) { C_above += sm.red64[w]; cnt_above += sm.red32[0][w]; }
    const unsigned int nb = nm;
    const unsigned long long guard = (unsigned long long)(KEY_NEG_INF + 1u) << 32;     // every finite element
    const unsigned long long cut_m = (unsigned long long)tk << 32;
    unsigned long long cutc = max(guard, cut_m);
    unsigned long long mass_in = 0ull;
    unsigned int n_in = 0u;
    bool chunks_final = true;                     // the per-chunk masses include the listed elements that are in
    if (listed && nb > 0u) {
        unsigned long long rest = max(target > C_above ? target - C_above : 1ull, 1ull);
        // Listed elements that are in for sure although they sit in the crossing bin (the medium path below finds
        // them above the sub-bin the cut falls into): their mass and number
        unsigned long long sure_mass = 0ull;
        unsigned int sure_n = 0u;
        bool small_ready = (nb <= (unsigned int)DENSE_THREADS && !overflow);
        unsigned int n_small = nb;
        uint32_t tie_v = 0u;                      // medium / crowded path: the cut falls among the ties of this key
        bool tie_path = false, in_smem = false, no_target = false;     // no_target: top-p does not decide inside the short list
        unsigned int tie_n = 0u;
        if (!small_ready && nb <= (unsigned int)MEMBER_CAP && !overflow) {
            // Medium path: up to MEMBER_CAP listed elements (low-precision logits: a few values, hundreds of ties
            // each).  One level of 512 sub-bins uniform over the listed keys' span separates the values; the
            // sub-bin the cut falls into then holds few elements (ranked like a short list) or the ties of one key.
            in_smem = true;
            const unsigned long long *gm = P.members + (size_t)row * MEMBER_CAP;
            for (int i = tid; i < (int)nb; i += DENSE_THREADS) dyn[i] = __ldcg(&gm[i]);
            const uint32_t kmin = __ldcg(&dr->kmin), kmax = __ldcg(&dr->kmax);
            const unsigned long long span = (unsigned long long)(kmax - kmin) + 1ull;
            unsigned int *scnt = sm.sub[0], *slo = sm.sub[1], *shi = sm.sub[2], *smin = sm.sub[3], *smax = sm.sub[4];
            scnt[tid] = 0u; slo[tid] = 0u; shi[tid] = 0u; smin[tid] = 0xFFFFFFFFu; smax[tid] = 0u;
            __syncthreads();
            const unsigned long long mult = ((unsigned long long)DENSE_THREADS << 32) / span;      // (no division per element)
            auto subbin = [=](uint32_t key) -> int { return min(DENSE_THREADS - 1, (int)(((unsigned long long)(key - kmin) * mult) >> 32)); };
            for (int i = tid; i < (int)nb; i += DENSE_THREADS) {
                const uint32_t key = (uint32_t)(dyn[i] >> 32);
                const int sb = subbin(key);
                const unsigned long long w1 = qweight(key, Mf);
                // lanes holding the same key (ties: same sub-bin, same weight) add once
                const unsigned int peers = __match_any_sync(__activemask(), key);
                if ((tid & 31) == __ffs(peers) - 1) {
                    const unsigned int np = __popc(peers);
                    const unsigned long long w = w1 * np;
                    atomicAdd(&scnt[sb], np);
                    const unsigned int lo = (unsigned int)w, hi = (unsigned int)(w >> 32);
                    unsigned int carry = 0;
                    if (lo) { const unsigned int old = atomicAdd(&slo[sb], lo); carry = (old + lo < old) ? 1u : 0u; }
                    if (hi + carry) atomicAdd(&shi[sb], hi + carry);
                    atomicMin(&smin[sb], key); atomicMax(&smax[sb], key);
                }
            }
            __syncthreads();
            // thread t owns sub-bin 511 - t (from the top): mass and number of the listed elements above it
            const int sbm = DENSE_THREADS - 1 - tid;
            const unsigned long long mmass = (unsigned long long)slo[sbm] | ((unsigned long long)shi[sbm] << 32);
            unsigned long long tot;
            const unsigned long long pre = dense_block_scan<unsigned long long>(mmass, sm.red64, tid, tot);
            const unsigned int mcnt = scnt[sbm];
            unsigned int cincl = mcnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const unsigned int up = __shfl_up_sync(0xFFFFFFFFu, cincl, o); if (lane >= o) cincl += up; }
            if (lane == 31) sm.red32[0][warp] = cincl;
            if (tid == 0) sm.flag = 0;
            __syncthreads();
            unsigned int coff = 0u;
            for (int w = 0; w < warp; ++w) coff += sm.red32[0][w];
            const unsigned int cpre = coff + cincl - mcnt;
            {
                // the sub-bin where the running mass reaches what is missing ...
                const unsigned long long r = min(rest, max(tot, 1ull));
                if (mmass > 0ull && pre < r && r <= pre + mmass) sm.flag = sbm;
            }
            __syncthreads();
            // ... against the sub-bin of the min-p threshold: the higher one decides (DENSE_THREADS: above every listed key)
            int xb = sm.flag;
            bool by_mass = true;
            if (tk) {
                const int sbt = (tk > kmax) ? DENSE_THREADS : (tk >= kmin ? subbin(tk) : -1);
                if (sbt > xb) { xb = sbt; by_mass = false; }
            }
            if (xb >= DENSE_THREADS) {
                // no listed element passes min-p: nothing of the bin is in
                small_ready = true; n_small = 0u; no_target = true;
                sm.comp[tid] = 0ull;
                __syncthreads();
            } else {
                if (sbm == xb) { sm.bc64[2] = pre; sm.cnt_above = cpre; }
                __syncthreads();
                sure_mass = sm.bc64[2];
                sure_n = sm.cnt_above;
                if (by_mass) rest = (rest > sure_mass) ? rest - sure_mass : 1ull; else no_target = true;
                const unsigned int cx = scnt[xb];
                const uint32_t xmin = smin[xb], xmax = smax[xb];
                __syncthreads();
            if (cx <= (unsigned int)DENSE_THREADS) {
                // gather the sub-bin's elements as the short list
                if (tid == 0) sm.nstage = 0u;
                sm.comp[tid] = 0ull;
                __syncthreads();
                for (int i = tid; i < (int)nb; i += DENSE_THREADS) {
                    const unsigned long long m = dyn[i];
                    if (subbin((uint32_t)(m >> 32)) == xb) sm.comp[atomicAdd(&sm.nstage, 1u)] = m;
                }
                __syncthreads();
                n_small = cx;
                small_ready = true;
            } else if (xmin == xmax) {
                tie_path = true; tie_v = xmin; tie_n = cx;
            } else {
                return false;
            }
            // the elements above the sub-bin are in: their mass goes to their tiles and chunks
            for (int i = tid; i < (int)nb; i += DENSE_THREADS) {
                const unsigned long long m = dyn[i];
                const uint32_t key = (uint32_t)(m >> 32);
                if (subbin(key) > xb && m >= cutc) {
                    const unsigned long long w = qweight(key, Mf);
                    const uint32_t idx = ~(uint32_t)m;
                    if (w) { smem_add_u64(&sm.tile_mass[idx / CTA_TILE], w); smem_add_u64(&sm.chunk[idx / DENSE_CHUNK], w); }
                }
            }
            __syncthreads();
            }
        } else if (!small_ready) {
            // a crowded bin: resolvable here only if it holds one value repeated (low-precision logits)
            const uint32_t kmin = __ldcg(&dr->kmin), kmax = __ldcg(&dr->kmax);
            if (kmin != kmax) return false;
            tie_path = true; tie_v = kmin; tie_n = nb;
        }
        if (small_ready) {
            // at most one listed element per thread: ranks by warp sorts and binary searches, then the running mass
            // in ranking order
            int rank;
            const unsigned long long key = rank_keys<DENSE_THREADS, BlockSync>(sm.comp, (int)n_small, tid, rank);
            const unsigned long long wk = key ? qweight((uint32_t)(key >> 32), Mf) : 0ull;
            __syncthreads();                      // every search has read the runs
            if (key) { sm.comp[rank] = key; sm.wt[rank] = wk; }
            if (tid == 0) { sm.bc64[0] = 0ull; sm.bc64[1] = 0ull; }
            __syncthreads();
            const bool have = (unsigned int)tid < n_small;
            const unsigned long long mine_c = have ? sm.comp[tid] : 0ull, mine_w = have ? sm.wt[tid] : 0ull;
            unsigned long long total_m;
            const unsigned long long pre = dense_block_scan<unsigned long long>(mine_w, sm.red64, tid, total_m);
            if (target && !no_target) {
                // the element at which the running mass first reaches what is still missing above it
                const unsigned long long r = min(rest, max(total_m, 1ull));
                if (mine_w > 0ull && pre < r && r <= pre + mine_w) sm.bc64[0] = mine_c;
                __syncthreads();
                cutc = max(cutc, sm.bc64[0]);
            }
            // what of the list is in: a prefix of the ranking; its mass goes to its tiles and chunks for the draw
            const bool inc = have && mine_c >= cutc;
            if (inc && mine_w) {
                const uint32_t idx = ~(uint32_t)mine_c;
                smem_add_u64(&sm.tile_mass[idx / CTA_TILE], mine_w);
                smem_add_u64(&sm.chunk[idx / DENSE_CHUNK], mine_w);
            }
            n_in = (unsigned int)__syncthreads_count(inc ? 1 : 0);
            if (have && (unsigned int)tid + 1u == n_in) sm.bc64[1] = pre + mine_w;
            __syncthreads();
            mass_in = (n_in ? sm.bc64[1] : 0ull) + sure_mass;
            n_in += sure_n;
        } else if (tie_path) {
            // the cut falls among tie_n elements of one key: the first m of them in index order are in
            chunks_final = false;
            const uint32_t v = tie_v;
            const unsigned long long wv = qweight(v, Mf);
            unsigned long long m = tie_n;
            if (tk && v < tk) m = 0ull;
            if (target && !no_target && m > 0ull && wv > 0ull) {
                const unsigned long long need = (rest + wv - 1ull) / wv;
                m = min(m, max(need, 1ull));
            }
            // ties per tile: from the row's tile records when the whole bin is this key, else counted from the list
            if (in_smem) {
                if (tid < MAX_TILES) sm.tile_nb[tid] = 0u;
                __syncthreads();
                for (int i = tid; i < (int)nb; i += DENSE_THREADS) {
                    const unsigned long long mm = dyn[i];
                    if ((uint32_t)(mm >> 32) == v) atomicAdd(&sm.tile_nb[(~(uint32_t)mm) / CTA_TILE], 1u);
                }
                __syncthreads();
            }
            int jt = -1;
            unsigned long long before = 0ull;
            if (m > 0ull && m < (unsigned long long)tie_n) {
                unsigned long long cum = 0ull;
                for (int j = 0; j < tiles; ++j) {
                    const unsigned long long t = sm.tile_nb[j];
                    if (jt < 0 && cum + t >= m) { jt = j; before = cum; }
                    cum += t;
                }
            }
            unsigned long long cut_v;
            if (m == 0ull) cut_v = ((unsigned long long)v + 1ull) << 32;
            else if (jt < 0) cut_v = (unsigned long long)v << 32;
            else {
                const int idx = dense_tile_find_tie(P, row, jt, v, m - 1ull - before, sm, tid);
                cut_v = ((unsigned long long)v << 32) | (uint32_t)(~(uint32_t)idx);
            }
            cutc = max(cutc, cut_v);
            __syncthreads();
            if (tid == 0) {
                unsigned long long left = m;
                for (int j = 0; j < tiles; ++j) {
                    const unsigned long long t = min(left, (unsigned long long)sm.tile_nb[j]);
                    sm.tile_mass[j] += t * wv;
                    left -= t;
                }
            }
            mass_in = m * wv + sure_mass;
            n_in = (unsigned int)m + sure_n;
            __syncthreads();
        }
    }
    const unsigned long long W = C_above + mass_in;
    const int support = (int)(cnt_above + n_in);
    const uint32_t a_acc = cells.x, a_draw = cells.y;
    uint32_t flags = F_DENSE;
    float p_draft = 0.0f;
    if (P.op == OP_VERIFY && c.l < P.K) {
        const int d = P.draft_tokens[(size_t)c.b * P.K + c.l];        // (the value the caller read; an id outside the vocabulary is reported as it is)
        unsigned long long qd = 0ull;
        double Q = 0.0;
        if (draft >= 0) {
            if ((((unsigned long long)key_draft << 32) | (uint32_t)(~(uint32_t)draft)) >= cutc) qd = qweight(key_draft, Mf);
            Q = (double)q_draft;
        }
        const double Pd = (double)qd / (double)W;
        const bool accept = (Pd > 0.0) && (cell_to_u(a_acc) * Q <= Pd);
        p_draft = (float)Pd;
        if (accept) {
            // the request moves on with the draft token: neither the residual nor a draw of this position is read
            if (tid == 0) emit_row(P, c, row, d, 0.0f, flags | F_ACCEPT, support, p_draft);
            return true;
        }
        // rejected: the residual pass finishes the position
        if (tid < tiles) dt[tid].mass = sm.tile_mass[tid];
        if (tid == 0) {
            dr->cutc = cutc; dr->W = W; dr->p_draft = p_draft; dr->support = support; dr->Mkey = Mkey;
            __threadfence();
            const unsigned int slot = atomicAdd(&P.error[WS_NRESID], 1u);
            P.rlist[slot] = row;
            dr->state = 2u;                                  // the residual draw's CTA of this row has work
        }
        return true;
    }
    // plain draw
    const unsigned long long T = draw_target(W, a_draw);
    if (chunks_final) {
        if (tid < 32) {
            unsigned long long qt;
            const int token = dense_warp_draw(P, row, tiles, sm, cutc, Mf, T, lane, qt);
            if (tid == 0) emit_row(P, c, row, token, (float)((double)qt / (double)W), flags, support, 0.0f);
        }
        return true;
    }
    // (slow paths above: the per-chunk masses are not final; tile-level CDF, then the element inside the tile)
    int jt = tiles - 1;
    unsigned long long before = 0ull;
    {
        unsigned long long cum = 0ull;
        bool hit = false;
        for (int j = 0; j < tiles; ++j) {
            const unsigned long long t = sm.tile_mass[j];
            if (!hit && t > 0ull && cum + t > T) { jt = j; before = cum; hit = true; }
            cum += t;
        }
        if (!hit) {                               // (T < W always; kept for safety: the last tile with mass)
            cum = 0ull;
            for (int j = 0; j < tiles; ++j) { if (sm.tile_mass[j] > 0ull) { jt = j; before = cum; } cum += sm.tile_mass[j]; }
        }
    }
    const unsigned long long cc = cutc;
    auto wf = [=](uint32_t key, int idx) -> unsigned long long {
        const unsigned long long wq = qweight(key, Mf);
        return ((((unsigned long long)key << 32) | (uint32_t)(~(uint32_t)idx)) >= cc) ? wq : 0ull;
    };
    unsigned long long qt = 0ull;
    const int token = dense_tile_find<unsigned long long>(P, row, jt, T - before, wf, sm.red64, sm, tid, qt);
    if (tid == 0) emit_row(P, c, row, token, (float)((double)qt / (double)W), flags, support, 0.0f);
    return true;
}

// Row-level parameters of a pass, derived by every CTA that needs them from what the earlier kernels left.
struct DenseRowPar {
    int kind;                                  // 0 nothing to do, 1 histogram items (pass H), 2 collect items (pass C)
    uint32_t Mkey, tk, klo, khi;
    unsigned long long target;
    float scale;
};

// What the streaming kernel left about a row, and what follows from it for the stage at hand.
//   stage 2: top-p rows take pass H; the others know their cut from the row maximum (min-p: the elements at or
//            above the threshold key; neither: every finite element - no bin, no list) and take pass C at once;
//   stage 3: top-p rows take pass C with the crossing bin found from the row's histogram (computed here, by every
//            CTA that meets the row; dyn holds the bins meanwhile);
//   stage 4 (the row's finish): top-p rows read what stage 3 stored, the others are as in stage 2.
// `first` marks the one CTA that speaks for the row (emits the rows without a token in stage 2, stores the cut in stage 3).
__device__ __forceinline__ DenseRowPar dense_row_par(const KParams &P, int row, int tiles, DenseShared &sm, unsigned long long *dyn, int tid,
                                                     const int stage, const bool first, RowCfg &c) {
    DenseRowPar r;
    r.kind = 0; r.tk = 0u; r.klo = 0u; r.khi = 0u; r.target = 0ull; r.scale = 0.0f;
    const CfgRaw raw = fetch_cfg(P, row);
    const DenseRow *dr = P.drow + row;
    uint32_t s_tk = 0u, s_klo = 0u, s_khi = 0u, s_state = 0u;
    unsigned long long s_target = 0ull;
    DenseBins bins;
    if (stage == 3) bins = dense_load_bins(P, row, tid);          // (only top-p rows use them; asked for before anything is waited for)
    if (stage == 4) { s_state = __ldcg(&dr->state); s_tk = __ldcg(&dr->tk); s_klo = __ldcg(&dr->klo); s_khi = __ldcg(&dr->khi); s_target = __ldcg(&dr->target); }
    dense_row_stats(P, row, tiles, sm, tid);
    __syncthreads();
    r.Mkey = sm.Mkey;
    const uint32_t mkey = sm.mkey;
    const unsigned int Nf = sm.Nf;
    bool bad = sm.bad != 0u;
    __syncthreads();
    c = resolve_cfg(P, row, raw);
    bad = bad || c.bad;
    if (bad || Nf == 0u) {
        if (stage == 2 && first && tid == 0) emit_row(P, c, row, -1, 0.0f, (bad ? F_BADPARAM : F_NO_TOKEN) | F_DENSE, 0, 0.0f);
    } else if (c.z & M_TOP_P) {
        if (stage == 2) {
            r.kind = 1; r.scale = dense_scale(r.Mkey, mkey, Nf);
        } else if (stage == 3) {
            const DenseCut cut = dense_hist_finish(P, c, row, sm, bins, tid, r.Mkey, dense_scale(r.Mkey, mkey, Nf), first);
            r.kind = 2; r.tk = cut.tk; r.klo = cut.klo; r.khi = cut.khi; r.target = cut.target;
        } else if (s_state == 1u) {
            r.kind = 2; r.tk = s_tk; r.klo = s_klo; r.khi = s_khi; r.target = s_target;
        }
    } else if (stage != 3) {
        r.kind = 2;
        r.tk = (c.z & M_MIN_P) ? minp_key(unkey(r.Mkey), c.theta) : 0u;
        r.klo = 0xFFFFFFFFu; r.khi = r.tk ? r.tk - 1u : KEY_NEG_INF;
    }
    return r;
}

// The item loop of stages 2 and 3: the (row, tile part) items of the call's rows of this class are dealt in
// contiguous ranges, so that a CTA's items mostly belong to one row whose parameters it derives once.  No CTA waits
// for another: the rows are finished in the kernel that follows (sonic_dense_finish_kernel).
__device__ __forceinline__ void dense_items(const KParams &P, int tiles, int cta, int ncta, unsigned long long *dyn, DenseShared &sm, const int stage) {
    const int tid = threadIdx.x;
    const int head = __ldcg(&P.dlist[tid & 31]);          // (the list's region holds 64 entries at least)
    const int nd = (int)__ldcg(&P.error[WS_NDENSE]);
    const int sub = dense_pick_sub(nd, tiles, ncta);
    const int per_row = tiles * sub;
    const DenseRange rg = dense_range(nd * per_row, cta, ncta);
    int cur_row = -1;
    DenseRowPar par;
    par.kind = 0;
    for (int item = rg.lo; item < rg.hi; ++item) {
        const DenseItem it = dense_item(P.dlist, head, item, tiles, sub);
        uint4 kv[DENSE_NV];
        dense_load_keys(P, it, tid, kv);
        if (it.row != cur_row) {
            cur_row = it.row;
            RowCfg c;
            par = dense_row_par(P, it.row, tiles, sm, dyn, tid, stage, it.tile == 0 && it.part == 0, c);
        }
        if (par.kind == 1) {
            unsigned int *hm0 = reinterpret_cast<unsigned int *>(dyn), *hm1 = hm0 + DBINS;
            dense_hist_item(P, it, kv, unkey(par.Mkey), par.scale, hm0, hm1, tid);
        } else if (par.kind == 2) {
            dense_collect_part(P, it, kv, unkey(par.Mkey), par.klo, par.khi, sm, dyn, tid);
        }
        __syncthreads();
    }
}

// Stage 2 never waits for its predecessor in the stream: on the library's internal stream it is an ordinary launch
// behind the streaming kernel; on the caller's stream it is a programmatic dependent of the merge kernel, whose CTAs
// let their dependents go only after their own wait for the streaming kernel, so when a CTA of this grid starts,
// the streaming kernel is complete and its results are visible.
__global__ void __launch_bounds__(DENSE_THREADS, 2)
sonic_dense_stage2_kernel(const KParams P, const int tiles) {
    extern __shared__ __align__(16) unsigned char dense_dyn_raw[];
    __shared__ DenseShared sm;
    pdl_launch_dependents();
    KERNEL_T0(6);
    dense_items(P, tiles, (int)blockIdx.x, (int)gridDim.x, reinterpret_cast<unsigned long long *>(dense_dyn_raw), sm, 2);
    KERNEL_T1(6);
}

__global__ void __launch_bounds__(DENSE_THREADS, 2)
sonic_dense_collect_kernel(const KParams P, const int tiles) {
    extern __shared__ __align__(16) unsigned char dense_dyn_raw[];
    __shared__ DenseShared sm;
    pdl_launch_dependents();
    pdl_wait_primary();
    KERNEL_T0(3);
    dense_items(P, tiles, (int)blockIdx.x, (int)gridDim.x, reinterpret_cast<unsigned long long *>(dense_dyn_raw), sm, 3);
    KERNEL_T1(3);
}

// The rows' finish, one CTA per row of the call (those of other classes leave at once): a programmatic dependent of
// pass C, whose completion is the only synchronisation a row needs.
__global__ void __launch_bounds__(DENSE_THREADS)
sonic_dense_finish_kernel(const KParams P, const int tiles) {
    extern __shared__ __align__(16) unsigned char dense_dyn_raw[];
    __shared__ DenseShared sm;
    unsigned long long *dyn = reinterpret_cast<unsigned long long *>(dense_dyn_raw);
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    // One CTA per row of the call: the row is known at launch, so its parameters are read - and the CTAs of rows of
    // other classes are gone - before the wait (inputs only; nothing here depends on the earlier kernels).
    const int row = blockIdx.x;
    {
        const RowCfg c0 = load_cfg(P, row);
        if (c0.cls != CLS_DENSE) return;
    }
    const int req = (P.op == OP_VERIFY) ? row / (P.K + 1) : row;
    const unsigned long long seed = P.seed ? P.seed[req] : 0ull, off = P.offset ? P.offset[req] : 0ull;
    // verification: the position's draft token and its draft probability (inputs)
    int draft = -1;
    float q_draft = 0.0f;
    if (P.op == OP_VERIFY) {
        const int l = row - req * (P.K + 1);
        if (l < P.K) {
            const int d = P.draft_tokens[(size_t)req * P.K + l];
            if (d >= 0 && d < P.V) { draft = d; q_draft = __ldg(P.draft_probs + ((size_t)req * P.K + l) * (size_t)P.V + d); }
        }
    }
    pdl_wait_primary();
    KERNEL_T0(8);
    {
        RowCfg c;
        const DenseRowPar par = dense_row_par(P, row, tiles, sm, dyn, tid, 4, false, c);
        if (__ldcg(&P.error[WS_ERROR]) & ERR_TIMEOUT) {       // (a wait of the streaming kernel ran out: the call's last kernel reports it for every row)
            KERNEL_T1(8);
            return;
        }
        if (par.kind != 0) {
            uint32_t r4[4];
            const unsigned long long pos = off + (unsigned long long)c.l;
            philox4x32_10((uint32_t)pos, (uint32_t)(pos >> 32), (uint32_t)c.b, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), r4);
            const uint2 cells = make_uint2(r4[0] >> 8, r4[1] >> 8);
            const bool ok = dense_finish(P, c, row, tiles, sm, dyn, tid, par.Mkey, par.klo <= par.khi, par.target, par.tk, cells, draft, q_draft);
            if (!ok && tid == 0) { P.rs[row].status = ST_FAILED; atomicAdd(&P.error[WS_FAILED_ROWS], 1u); }
        }
    }
    KERNEL_T1(8);
}

// Stage 4 (verification calls): the residual max(0, p - q) of the positions whose draft was rejected.  The
// support's total weight W is known here only in fixed point (relative error up to 1e-7 on peaked rows, too
// coarse where p - q cancels), so an item accumulates, in fp64, the residual sum R~ taken with that W~, the sum Pp of
// the weights whose residual is positive, and the plain sum S of the weights; with W = sum of S the row's finish
// corrects each tile's residual to R~ - (1/W~ - 1/W) * Pp (exact up to the elements whose residual changes
// sign between W~ and W, each of which contributes less than 1e-7 of its own probability).
// Weights: an element that carries more than 2^-7 of the support's mass (at most 128 per row, usually a handful) is
// weighed with the fp64 exponential: its residual is a difference of two numbers of that size.  The others use an
// fp32 exponential of relative error below 1e-7 with no bias; independent errors of that size on probabilities
// below 2^-7 add up to less than 1e-8 in the cumulative sums.
// The draft's probabilities of 16 consecutive elements (first a multiple of 16), independent of the keys: an element
// outside the support has weight 0 and so a residual <= 0 whatever q is; indices past the row's end are clamped.
__device__ __forceinline__ void resid_load_q(const float *q, int first, int V, float (&qv)[DENSE_EPT]) {
    if (first + DENSE_EPT <= V && ((reinterpret_cast<uintptr_t>(q + first) & 15) == 0)) {
        const float4 *s4 = reinterpret_cast<const float4 *>(q + first);
#pragma unroll
        for (int k = 0; k < DENSE_NV; ++k) {
            const float4 v = __ldg(s4 + k);
            qv[4 * k] = v.x; qv[4 * k + 1] = v.y; qv[4 * k + 2] = v.z; qv[4 * k + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int e = 0; e < DENSE_EPT; ++e) qv[e] = __ldg(q + min(first + e, V - 1));
    }
}

__device__ __forceinline__ double resid_weight(uint32_t key, float Mf, double Md, float big) {
    const float y = unkey(key);
    const float w32 = exp_accurate(__fsub_rn(y, Mf));
    return (w32 > big) ? exp((double)y - Md) : (double)w32;
}

// The element of one tile at which the running sum of the residuals first exceeds `rest` (the tile's last element of
// positive residual if rounding keeps the sum below it; -1 if the tile has none).  Whole CTA; a thread holds its 16
// residuals in registers.
__device__ int resid_tile_find(const KParams &P, int row, int tile, const float *q, unsigned long long cutc, float Mf, double Md,
                               float big, double inv_W, double rest, DenseShared &sm, int tid) {
    const int first = tile * CTA_TILE + tid * DENSE_EPT;
    const uint4 *src = reinterpret_cast<const uint4 *>(P.ykeys + (size_t)row * ((size_t)P.ytiles * CTA_TILE) + first);
    uint4 kv[DENSE_NV];
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) kv[k] = src[k];
    float qv[DENSE_EPT];
    resid_load_q(q, first, P.V, qv);
    if (tid == 0) { sm.flag = -1; sm.digit = -1; }
    double r[DENSE_EPT];
    double s = 0.0;
    int lastpos = -1;
#pragma unroll
    for (int k = 0; k < DENSE_NV; ++k) {
        const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = 4 * k + u;
            const bool in = (((unsigned long long)key4[u] << 32) | (uint32_t)(~(uint32_t)(first + e))) >= cutc;
            const double w = in ? resid_weight(key4[u], Mf, Md, big) : 0.0;
            const double v = w * inv_W - (double)qv[e];
            r[e] = v > 0.0 ? v : 0.0;
            s += r[e];
            if (v > 0.0) lastpos = first + e;
        }
    }
    double total;
    const double pre = dense_block_scan<double>(s, sm.redd[0], tid, total);
    if (s > 0.0 && pre <= rest && rest < pre + s) {
        double cum = pre;
        int found = -1;
#pragma unroll
        for (int e = 0; e < DENSE_EPT; ++e) {
            cum += r[e];
            if (r[e] > 0.0 && found < 0 && cum > rest) found = first + e;
        }
        sm.flag = found < 0 ? lastpos : found;
    }
    __syncthreads();
    if (sm.flag < 0) {
        if (lastpos >= 0) atomicMax(&sm.digit, lastpos);
        __syncthreads();
        if (tid == 0) sm.flag = sm.digit;
        __syncthreads();
    }
    const int res = sm.flag;
    __syncthreads();
    return res;
}

// One CTA's items: contiguous ranges over the rows of the residual list, a tile per item.
__global__ void __launch_bounds__(DENSE_THREADS, 2)
sonic_dense_resid_kernel(const KParams P, const int tiles) {
    __shared__ DenseShared sm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    pdl_wait_primary();
    KERNEL_T0(4);
    const int head = __ldcg(&P.rlist[tid & 31]);
    const int nr = (int)__ldcg(&P.error[WS_NRESID]);
    const DenseRange rg = dense_range(nr * tiles, (int)blockIdx.x, (int)gridDim.x);
    int cur_row = -1;
    unsigned long long cutc = 0ull;
    float Mf = 0.0f, big = 0.0f;
    double Md = 0.0, inv_Wt = 0.0;
    const float *q = nullptr;
    for (int item = rg.lo; item < rg.hi; ++item) {
        const DenseItem it = dense_item(P.rlist, head, item, tiles, 1);
        const int row = it.row, tile = it.tile;
        uint4 kv[DENSE_NV];
        dense_load_keys(P, it, tid, kv);
        {
            const int b = row / (P.K + 1), l = row - b * (P.K + 1);
            q = P.draft_probs + ((size_t)b * P.K + l) * (size_t)P.V;
        }
        float qv[DENSE_EPT];
        resid_load_q(q, tile * CTA_TILE + tid * DENSE_EPT, P.V, qv);
        if (row != cur_row) {
            cur_row = row;
            const DenseRow *dr = P.drow + row;
            cutc = __ldcg(&dr->cutc);
            const unsigned long long Wq = __ldcg(&dr->W);
            Mf = unkey(__ldcg(&dr->Mkey));
            Md = (double)Mf;
            inv_Wt = 1099511627776.0 / (double)Wq;                      // 1 / W~
            big = (float)((double)Wq * (1.0 / 1099511627776.0) * (1.0 / 128.0));
        }
        double R = 0.0, Pp = 0.0, S = 0.0;
#pragma unroll
        for (int k = 0; k < DENSE_NV; ++k) {
            const uint32_t key4[4] = {kv[k].x, kv[k].y, kv[k].z, kv[k].w};
            const int base_idx = tile * CTA_TILE + tid * DENSE_EPT + 4 * k;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = base_idx + u;
                const bool in = (((unsigned long long)key4[u] << 32) | (uint32_t)(~(uint32_t)idx)) >= cutc;
                const double w = in ? resid_weight(key4[u], Mf, Md, big) : 0.0;
                const double r = w * inv_Wt - (double)qv[4 * k + u];
                S += w;
                R += (r > 0.0) ? r : 0.0;
                Pp += (r > 0.0) ? w : 0.0;
            }
        }
        // fixed reduction order: lanes by butterfly, warps in order
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            R += __shfl_xor_sync(0xFFFFFFFFu, R, off);
            Pp += __shfl_xor_sync(0xFFFFFFFFu, Pp, off);
            S += __shfl_xor_sync(0xFFFFFFFFu, S, off);
        }
        if (lane == 0) { sm.redd[0][warp] = R; sm.redd[1][warp] = Pp; sm.redd[2][warp] = S; }
        __syncthreads();
        if (tid == 0) {
            double r = 0.0, p = 0.0, s = 0.0;
            for (int w = 0; w < DENSE_WARPS; ++w) { r += sm.redd[0][w]; p += sm.redd[1][w]; s += sm.redd[2][w]; }
            DenseTile *dt = P.dtile + (size_t)row * MAX_TILES + tile;
            dt->R = r; dt->Pp = p; dt->S = s;
        }
        __syncthreads();
    }
    KERNEL_T1(4);
}

// The residual draw, one CTA per row of the residual list (a programmatic dependent of the kernel above).
__global__ void __launch_bounds__(DENSE_THREADS)
sonic_dense_resid_finish_kernel(const KParams P, const int tiles) {
    __shared__ DenseShared sm;
    const int tid = threadIdx.x;
    pdl_launch_dependents();
    // one CTA per row of the call, as in the rows' finish: rows of other classes, and positions without a draft, leave
    // before the wait; rows whose draft was accepted right after it
    const int row = blockIdx.x;
    {
        const RowCfg c0 = load_cfg(P, row);
        if (c0.cls != CLS_DENSE || c0.l >= P.K) return;
    }
    pdl_wait_primary();
    KERNEL_T0(9);
    if (__ldcg(&(P.drow + row)->state) == 2u) {
        DenseRow *dr = P.drow + row;
        DenseTile *dt = P.dtile + (size_t)row * MAX_TILES;
        const RowCfg c = load_cfg(P, row);
        const unsigned long long cutc = __ldcg(&dr->cutc), Wq = __ldcg(&dr->W);
        const uint32_t Mkey = __ldcg(&dr->Mkey);
        const float Mf = unkey(Mkey);
        const double Md = (double)Mf;
        const double inv_Wt = 1099511627776.0 / (double)Wq;
        const float big = (float)((double)Wq * (1.0 / 1099511627776.0) * (1.0 / 128.0));
        const float *q = P.draft_probs + ((size_t)c.b * P.K + c.l) * (size_t)P.V;
        uint32_t a_acc, a_draw;
        draw_cells(P, c, a_acc, a_draw);
        if (tid < 32) {
            // a tile's three sums per lane (one round of loads), added up in tile order by every lane alike
            double sj = 0.0, rj0 = 0.0, pj = 0.0;
            if (tid < tiles) { sj = __ldcg(&dt[tid].S); rj0 = __ldcg(&dt[tid].R); pj = __ldcg(&dt[tid].Pp); }
            double Wd = 0.0;
            for (int j = 0; j < tiles; ++j) Wd += __shfl_sync(0xFFFFFFFFu, sj, j);
            const double corr = inv_Wt - 1.0 / Wd;
            double rj = rj0 - corr * pj;
            rj = (tid < tiles && rj > 0.0) ? rj : 0.0;
            reinterpret_cast<double *>(sm.wt)[tid] = rj;
            double Rtot = 0.0;
            for (int j = 0; j < tiles; ++j) Rtot += __shfl_sync(0xFFFFFFFFu, rj, j);
            if (tid == 0) { sm.bcd[0] = Wd; sm.bcd[1] = Rtot; }
        }
        __syncthreads();
        const double Wd = sm.bcd[0], Rtot = sm.bcd[1];
        int token = -1;
        if (Rtot > 0.0) {
            const double target = cell_to_u(a_draw) * Rtot;
            const double *rj = reinterpret_cast<const double *>(sm.wt);
            int jt = -1;
            double before = 0.0, cum = 0.0;
            for (int j = 0; j < tiles; ++j) {
                if (jt < 0 && rj[j] > 0.0 && cum + rj[j] > target) { jt = j; before = cum; }
                cum += rj[j];
            }
            if (jt < 0) { cum = 0.0; for (int j = 0; j < tiles; ++j) { if (rj[j] > 0.0) { jt = j; before = cum; } cum += rj[j]; } }
            const double inv_Wd = 1.0 / Wd;
            __syncthreads();
            if (jt >= 0) token = resid_tile_find(P, row, jt, q, cutc, Mf, Md, big, inv_Wd, target - before, sm, tid);
        }
        if (token < 0) {
            // empty residual (p <= q on the whole support, by rounding): draw from p itself
            const unsigned long long T = draw_target(Wq, a_draw);
            int jt = tiles - 1;
            unsigned long long before = 0ull, cum = 0ull;
            bool hit = false;
            for (int j = 0; j < tiles; ++j) {
                const unsigned long long t = __ldcg(&dt[j].mass);
                if (!hit && t > 0ull && cum + t > T) { jt = j; before = cum; hit = true; }
                cum += t;
            }
            auto wf = [=](uint32_t key, int idx) -> unsigned long long {
                const unsigned long long wq = qweight(key, Mf);
                return ((((unsigned long long)key << 32) | (uint32_t)(~(uint32_t)idx)) >= cutc) ? wq : 0ull;
            };
            unsigned long long qt;
            __syncthreads();
            token = dense_tile_find<unsigned long long>(P, row, jt, T - before, wf, sm.red64, sm, tid, qt);
        }
        if (tid == 0) emit_row(P, c, row, token, 0.0f, F_DENSE, __ldcg(&dr->support), __ldcg(&dr->p_draft));
        __syncthreads();
    }
    KERNEL_T1(9);
}

}  // namespace sonic
