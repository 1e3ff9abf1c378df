// Exact full-vocabulary kernel: one thread-block cluster of 8 CTAs per row keeps
// the whole processed row resident in distributed shared memory (ordered 32-bit
// keys, 32768 per CTA) and answers any truncation exactly with radix descents
// over count / probability-mass histograms, cluster-wide reductions going
// through DSMEM and hardware cluster barriers (no flags, no spinning).
//
// It is the last resort of a call: (a) rows with a top-k beyond what the
// streaming path sorts, (b) rows the streaming path could not prove, (c) rows
// of the histogram path whose crossing bin was too crowded.  Usually there is
// none and the kernel returns at once.  (Rows with top-k off are finished by the
// histogram passes, sonic_dense.cuh.)  The paper bounds k at 128 and is lossy
// beyond it (Section 3.3); this path and the histogram path remove that bound.
//
// Probability mass is accumulated as 64-bit fixed point (2^-40 units of the
// largest weight), so sums are order-independent and replays are bit-identical.
#pragma once
#include <cooperative_groups.h>
#include "sonic_common.cuh"
#include "sonic_stream.cuh"

namespace sonic {
namespace cg = cooperative_groups;

constexpr int EX_THREADS = 512;
constexpr int EX_WARPS = EX_THREADS / 32;
constexpr int CL = 8;                         // CTAs per cluster
constexpr int SLICE_MAX = MAX_VOCAB / CL;     // 32768 keys per CTA
constexpr int HBINS = 2048;
constexpr int XV = 4;                         // 64-bit values per exchange

struct Cut {                                  // member: key > v || (key == v && index <= idx)
    uint32_t v;
    int idx;
};
__device__ __forceinline__ bool member(const Cut &c, uint32_t key, int gidx) {
    return key > c.v || (key == c.v && gidx <= c.idx);
}
__device__ __forceinline__ bool tighter(const Cut &a, const Cut &b) {   // a keeps fewer elements than b
    return a.v > b.v || (a.v == b.v && a.idx < b.idx);
}

constexpr int ORD_GROUPS = SLICE_MAX / EX_WARPS / 128;     // groups of 128 elements in a warp's run, at most
struct ExactShared {
    unsigned long long xch[2][CL][XV];
    unsigned long long vals[XV];
    unsigned long long wtot[EX_WARPS];
    unsigned long long wcnt[EX_WARPS];
    unsigned long long gtot[EX_WARPS][ORD_GROUPS];   // ordered passes: totals of each warp's groups of 128 elements
    unsigned long long red_mass[HBINS / CL];
    unsigned int red_cnt[HBINS / CL];
    unsigned int ucount;
    int flag;
    int ticket;                                      // the ordinal of the cluster's next row
};

struct ExactCtx {
    ExactShared *sh;
    uint32_t *keys;
    unsigned int *hcnt, *hm0, *hm1;            // per-bin count and 64-bit mass as two 32-bit words (32-bit adds, explicit carry)
    int rank, lo, len, per, tid, lane, warp;
    int phase;
    float Mf;                                  // largest processed logit
    float scale, inv_scale;                    // histogram bins per logit unit (a power of two) and its reciprocal
};

// All CTAs contribute XV values; afterwards every CTA holds all of them.
__device__ __forceinline__ void allgather(ExactCtx &x, const unsigned long long (&v)[XV],
                                          unsigned long long (&out)[CL][XV]) {
    __syncthreads();
    if (x.tid == 0) {
#pragma unroll
        for (int i = 0; i < XV; ++i) x.sh->vals[i] = v[i];
    }
    __syncthreads();
    if (x.tid < CL * XV) {
        int r = x.tid / XV, i = x.tid % XV;
        ExactShared *remote = cg::this_cluster().map_shared_rank(x.sh, r);
        remote->xch[x.phase][x.rank][i] = x.sh->vals[i];
    }
    cg::this_cluster().sync();
#pragma unroll
    for (int r = 0; r < CL; ++r)
#pragma unroll
        for (int i = 0; i < XV; ++i) out[r][i] = x.sh->xch[x.phase][r][i];
    x.phase ^= 1;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    return v;
}

// Sum over the block of one 64-bit value per thread; result valid in every thread.
__device__ __forceinline__ unsigned long long block_sum_u64(ExactCtx &x, unsigned long long v) {
    v = warp_sum_u64(v);
    __syncthreads();
    if (x.lane == 0) x.sh->wtot[x.warp] = v;
    __syncthreads();
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < EX_WARPS; ++w) t += x.sh->wtot[w];
    return t;
}

// Position for an element a lane wants to append to a list whose length lives in shared
// memory: one atomic per warp.  Every lane of the warp must call it (want = false to skip).
__device__ __forceinline__ unsigned int warp_append(unsigned int *counter, bool want, int lane) {
    const unsigned int m = __ballot_sync(0xFFFFFFFFu, want);
    unsigned int base = 0;
    if (lane == 0 && m) base = atomicAdd(counter, (unsigned int)__popc(m));
    base = __shfl_sync(0xFFFFFFFFu, base, 0);
    return base + __popc(m & ((1u << lane) - 1u));
}

// Ordered passes: elements are visited in vocabulary-index order (warp w owns a
// contiguous run of the slice, lanes interleaved), each with weight wf(local index)
// of a 64-bit type T (fixed-point mass, a count, or fp64).
template <typename T>
struct OrderedState {
    T cta_off;            // sum over the CTAs before this one
    T warp_off;           // sum over this CTA's warps before this warp
    T total;              // row total
    T cta_tot[CL];        // per-CTA totals
};

// Row total of wf (and of the 0/1 indicator cf, returned in count_out); leaves the per-warp totals of wf in
// shared memory for a following ordered_find.  One cluster barrier.
template <typename T, typename WF, typename CF>
__device__ void ordered_totals(ExactCtx &x, WF wf, CF cf, OrderedState<T> &st, unsigned long long &count_out) {
    const int wch = x.per / EX_WARPS;                    // elements per warp (multiple of 32)
    const int wlo = x.warp * wch;
    const int lane = x.lane;
    unsigned long long *gt = x.sh->gtot[x.warp];
    T wt = T(0);
    unsigned long long cn = 0;
    int g = 0;
    for (int i = wlo + lane; i < wlo + wch; i += 128, ++g) {      // four independent elements per trip
        T w4[4];
        unsigned long long c4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int ii = i + 32 * u;
            const bool in = ii < wlo + wch;
            w4[u] = in ? wf(ii) : T(0);
            c4[u] = in ? cf(ii) : 0ull;
        }
        // the trip's 128 consecutive elements form one group: its total is kept for ordered_find, and the warp
        // total is the sum of the group totals in order (every lane computes the same values)
        T ts = (w4[0] + w4[1]) + (w4[2] + w4[3]);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ts += __shfl_xor_sync(0xFFFFFFFFu, ts, off);
        if (lane == 0) gt[g] = *reinterpret_cast<unsigned long long *>(&ts);
        wt += ts;
#pragma unroll
        for (int u = 0; u < 4; ++u) cn += c4[u];
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cn += __shfl_xor_sync(0xFFFFFFFFu, cn, off);
    __syncthreads();
    if (x.lane == 0) { x.sh->wtot[x.warp] = *reinterpret_cast<unsigned long long *>(&wt); x.sh->wcnt[x.warp] = cn; }
    __syncthreads();
    T cta_total = T(0);
    unsigned long long cta_cnt = 0;
    st.warp_off = T(0);
    for (int w = 0; w < EX_WARPS; ++w) {
        const T v = *reinterpret_cast<T *>(&x.sh->wtot[w]);
        if (w == x.warp) st.warp_off = cta_total;
        cta_total += v;
        cta_cnt += x.sh->wcnt[w];
    }
    unsigned long long v[XV] = {*reinterpret_cast<unsigned long long *>(&cta_total), cta_cnt, 0, 0};
    unsigned long long all[CL][XV];
    allgather(x, v, all);
    st.total = T(0);
    st.cta_off = T(0);
    count_out = 0;
    for (int r = 0; r < CL; ++r) {
        const T t = *reinterpret_cast<T *>(&all[r][0]);
        st.cta_tot[r] = t;
        if (r == x.rank) st.cta_off = st.total;
        st.total += t;
        count_out += all[r][1];
    }
}

// First element (index order) whose inclusive running sum of wf exceeds `target`; uses the warp totals left by
// ordered_totals for the same wf.  Returns its global index (-1 if none) and its weight, in every CTA.  One
// cluster barrier.
template <typename T, typename WF>
__device__ int ordered_find(ExactCtx &x, T target, WF wf, const OrderedState<T> &st, T &weight_out) {
    const int wch = x.per / EX_WARPS;
    const int wlo = x.warp * wch;
    int cross_rank = -1;
    {
        T acc = T(0);
        for (int r = 0; r < CL; ++r) {
            if (cross_rank < 0 && acc + st.cta_tot[r] > target) cross_rank = r;
            acc += st.cta_tot[r];
        }
    }
    if (cross_rank == x.rank) {
        int cross_warp = -1;
        T acc = st.cta_off;
        for (int w = 0; w < EX_WARPS; ++w) {
            const T v2 = *reinterpret_cast<T *>(&x.sh->wtot[w]);
            if (cross_warp < 0 && acc + v2 > target) cross_warp = w;
            acc += v2;
        }
        if (cross_warp < 0) cross_warp = EX_WARPS - 1;    // rounding between levels
        if (x.warp == cross_warp) {
            const int lane = x.lane, lo_g = x.lo;
            T run = st.cta_off + st.warp_off;
            int found = -1, last_member = -1;
            T fw = T(0), lw = T(0);
            // First pass: skip the groups of 128 elements that end before the target (their totals were left by
            // ordered_totals).  Should rounding leave it without any positive element, a second pass scans the
            // whole run.
            for (int pass = 0; pass < 2 && found < 0 && last_member < 0; ++pass) {
                int istart = wlo;
                run = st.cta_off + st.warp_off;
                if (pass == 0) {
                    const int ngroups = (wch + 127) / 128;
                    T acc = run;
                    for (int gg = 0; gg + 1 < ngroups; ++gg) {      // never past the last group
                        const T t = *reinterpret_cast<T *>(&x.sh->gtot[x.warp][gg]);
                        if (acc + t > target) break;
                        acc += t;
                        istart += 128;
                    }
                    run = acc;
                }
                for (int i = istart; i < wlo + wch; i += 32) {
                    const T wv = wf(i + lane);
                    T incl = wv;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const T up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                        if (lane >= o) incl += up;
                    }
                    const unsigned int hit = __ballot_sync(0xFFFFFFFFu, (run + incl > target) && (wv > T(0)));
                    const unsigned int pos = __ballot_sync(0xFFFFFFFFu, wv > T(0));
                    if (hit) {
                        const int l = __ffs(hit) - 1;
                        found = lo_g + i + l;
                        fw = __shfl_sync(0xFFFFFFFFu, wv, l);
                        break;
                    }
                    if (pos) {
                        const int l = 31 - __clz(pos);
                        last_member = lo_g + i + l;
                        lw = __shfl_sync(0xFFFFFFFFu, wv, l);
                    }
                    run += __shfl_sync(0xFFFFFFFFu, incl, 31);
                }
            }
            if (found < 0) { found = last_member; fw = lw; }   // rounding between levels: last positive element
            if (x.lane == 0) { x.sh->flag = found; x.sh->vals[3] = *reinterpret_cast<unsigned long long *>(&fw); }
        }
    }
    __syncthreads();
    unsigned long long v2[XV] = {0, 0, 0, 0};
    if (cross_rank == x.rank) { v2[0] = (unsigned long long)(long long)x.sh->flag; v2[1] = x.sh->vals[3]; }
    unsigned long long all[CL][XV];
    allgather(x, v2, all);
    weight_out = T(0);
    if (cross_rank < 0) return -1;
    weight_out = *reinterpret_cast<T *>(&all[cross_rank][1]);
    return (int)(long long)all[cross_rank][0];
}

// One histogram level of a selection.  digit(key) gives the element's bin
// (larger bin = ranks earlier) or -1 if the element is outside the level's
// range; only members of `base` take part.  Scanning bins from the top, finds
// the bin where the running count (or mass) first reaches `target`; on return
// `target` is what is still needed inside that bin and `in_bin` is the bin's
// element count.  For by_mass with first == true the target is set to
// ceil(p * total mass) first.  Two cluster barriers.
template <typename DF>
__device__ int hist_level(ExactCtx &x, const Cut &base, bool by_mass, bool first, float p, int nbins, DF digit,
                          unsigned long long &target, unsigned long long &in_bin, unsigned long long *stg) {
    for (int i = x.tid; i < nbins; i += EX_THREADS) { x.hcnt[i] = 0; x.hm0[i] = 0; x.hm1[i] = 0; }
    __syncthreads();
    // four elements per thread and trip: their keys, bins and weights are computed first (independent chains
    // that overlap), then added to the histogram
    // The mass of a bin is a 64-bit integer kept as two 32-bit words: the low word takes one atomic add whose
    // returned old value reveals a carry; the high word is touched only on a carry or by weights >= 2^-8.
    // local copies of what the element loop reads (the context and the cut arrive by reference: read through them,
    // every access would go to memory)
    const uint32_t *keys = x.keys;
    unsigned int *hcnt = x.hcnt, *hm0 = x.hm0, *hm1 = x.hm1;
    const int len = x.len, lo_g = x.lo, per = x.per, tid = x.tid, lane = x.lane;
    const float Mf = x.Mf;
    const Cut bs = base;
    auto add_mass = [=](int b, unsigned long long q) {
        const unsigned int lo = (unsigned int)q, hi = (unsigned int)(q >> 32);
        unsigned int carry = 0;
        if (lo) { const unsigned int old = atomicAdd(&hm0[b], lo); carry = (old + lo < old) ? 1u : 0u; }
        if (hi + carry) atomicAdd(&hm1[b], hi + carry);
    };
    for (int i0 = 0; i0 < per; i0 += 4 * EX_THREADS) {
        int bin[4];
        unsigned long long q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = i0 + u * EX_THREADS + tid;
            bin[u] = -1; q[u] = 0ull;
            if (i < len) {
                const uint32_t key = keys[i];
                if (member(bs, key, lo_g + i)) {
                    bin[u] = digit(key);
                    if (by_mass && bin[u] >= 0) q[u] = qweight(key, Mf);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const unsigned int active = __ballot_sync(0xFFFFFFFFu, bin[u] >= 0);
            if (bin[u] < 0) continue;
            int same;
            __match_all_sync(active, bin[u], &same);
            if (same) {                               // the whole warp hits one bin: one lane adds for all
                const unsigned int n = __popc(active);
                unsigned long long qs = q[u];
                if (by_mass) {                        // 20-bit pieces: 32 of them sum below 2^25
                    const unsigned int p0 = __reduce_add_sync(active, (unsigned int)(q[u] & 0xFFFFFu));
                    const unsigned int p1 = __reduce_add_sync(active, (unsigned int)((q[u] >> 20) & 0xFFFFFu));
                    const unsigned int p2 = __reduce_add_sync(active, (unsigned int)(q[u] >> 40));
                    qs = (unsigned long long)p0 + ((unsigned long long)p1 << 20) + ((unsigned long long)p2 << 40);
                }
                if ((int)(__ffs(active) - 1) == lane) {
                    atomicAdd(&hcnt[bin[u]], n);
                    if (by_mass) add_mass(bin[u], qs);
                }
            } else {
                atomicAdd(&hcnt[bin[u]], 1u);
                if (by_mass) add_mass(bin[u], q[u]);
            }
        }
    }
    cg::this_cluster().sync();
    // CTA r reduces bins [r*bpr, (r+1)*bpr) over the cluster.  Remote shared-memory reads are slow, so
    // all of them are issued at once: thread t fetches (bin, rank) pairs t, t + EX_THREADS, ... into a
    // local staging area (the sort buffer, idle during histogram levels), then the owners add locally.
    const int bpr = nbins / CL;
    unsigned int *stg_cnt = reinterpret_cast<unsigned int *>(stg);                    // [CL][bpr]
    unsigned long long *stg_mass = stg + (CL * (HBINS / CL)) / 2;                       // [CL][bpr]
    {
        constexpr int TRIPS = (CL * (HBINS / CL) + EX_THREADS - 1) / EX_THREADS;       // 4
        unsigned int cc[TRIPS], a0[TRIPS], a1[TRIPS], a2[TRIPS];
#pragma unroll
        for (int u = 0; u < TRIPS; ++u) {
            const int pair = x.tid + u * EX_THREADS;
            const int r = pair / bpr, bl = pair - r * bpr;
            cc[u] = a0[u] = a1[u] = a2[u] = 0;
            if (r < CL) {
                const int bin = x.rank * bpr + bl;
                cc[u] = *cg::this_cluster().map_shared_rank(&x.hcnt[bin], r);
                if (by_mass) {
                    a0[u] = *cg::this_cluster().map_shared_rank(&x.hm0[bin], r);
                    a1[u] = *cg::this_cluster().map_shared_rank(&x.hm1[bin], r);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < TRIPS; ++u) {
            const int pair = x.tid + u * EX_THREADS;
            const int r = pair / bpr, bl = pair - r * bpr;
            if (r < CL) {
                stg_cnt[r * bpr + bl] = cc[u];
                stg_mass[r * bpr + bl] = (unsigned long long)a0[u] | ((unsigned long long)a1[u] << 32);
            }
        }
    }
    __syncthreads();
    unsigned long long sc = 0, sm = 0;
    if (x.tid < bpr) {
        unsigned int cc = 0;
        unsigned long long mm = 0;
#pragma unroll
        for (int r = 0; r < CL; ++r) { cc += stg_cnt[r * bpr + x.tid]; mm += stg_mass[r * bpr + x.tid]; }
        x.sh->red_cnt[x.tid] = cc;
        x.sh->red_mass[x.tid] = mm;
        sc = cc; sm = mm;
    }
    sc = block_sum_u64(x, sc);
    sm = block_sum_u64(x, sm);
    unsigned long long v[XV] = {sc, sm, 0, 0};
    unsigned long long all[CL][XV];
    allgather(x, v, all);                      // every remote histogram read precedes this barrier
    if (by_mass && first) {
        unsigned long long Zq = 0;
        for (int r = 0; r < CL; ++r) Zq += all[r][1];
        double t = ceil((double)p * (double)Zq);
        target = (unsigned long long)t;
        if (target > Zq) target = Zq;
        if (target < 1) target = 1;
    }
    // segment (CTA) holding the crossing, scanning from the top
    int seg = -1;
    unsigned long long cum = 0;
    for (int r = CL - 1; r >= 0; --r) {
        unsigned long long sseg = by_mass ? all[r][1] : all[r][0];
        if (cum + sseg >= target) { seg = r; break; }
        cum += sseg;
    }
    if (seg < 0) {                             // target beyond the total: cannot happen for valid calls
        seg = 0;
        cum -= by_mass ? all[0][1] : all[0][0];
        target = cum + (by_mass ? all[0][1] : all[0][0]);
    }
    // every CTA reads the crossing segment's reduced bins from their owner and scans them itself
    const unsigned int *rc = cg::this_cluster().map_shared_rank(&x.sh->red_cnt[0], seg);
    const unsigned long long *rm = cg::this_cluster().map_shared_rank(&x.sh->red_mass[0], seg);
    if (x.tid < 32) {
        // warp 0: lanes take bins from the top in chunks of 32; all remote reads are issued before the scan
        constexpr int CH = (HBINS / CL) / 32;        // 8 chunks at most
        unsigned long long pv[CH];
        unsigned int pc[CH];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
            const int t = bpr - 1 - ch * 32 - x.lane;
            pv[ch] = 0; pc[ch] = 0;
            if (t >= 0) { pc[ch] = rc[t]; pv[ch] = by_mass ? rm[t] : (unsigned long long)pc[ch]; }
        }
        unsigned long long c2 = cum;
        int found = -1;
        unsigned long long rest = 0, cnt = 0;
#pragma unroll
        for (int ch = 0; ch < CH; ++ch) {
            const int top = bpr - 1 - ch * 32;
            if (top < 0 || found >= 0) continue;
            const int t = top - x.lane;
            const unsigned long long val = pv[ch];
            const unsigned int cval = pc[ch];
            unsigned long long incl = val;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (x.lane >= o) incl += up;
            }
            unsigned int hit = __ballot_sync(0xFFFFFFFFu, t >= 0 && c2 + incl >= target);
            if (hit) {
                const int l = __ffs(hit) - 1;
                found = top - l;
                rest = target - (c2 + __shfl_sync(0xFFFFFFFFu, incl, l) - __shfl_sync(0xFFFFFFFFu, val, l));
                cnt = __shfl_sync(0xFFFFFFFFu, cval, l);
            } else {
                c2 += __shfl_sync(0xFFFFFFFFu, incl, 31);
            }
        }
        if (found < 0) { found = 0; rest = 1; cnt = rc[0]; }
        if (x.lane == 0) {
            x.sh->vals[0] = (unsigned long long)(seg * bpr + found);
            x.sh->vals[1] = rest;
            x.sh->vals[2] = cnt;
        }
    }
    __syncthreads();
    const int bin = (int)x.sh->vals[0];
    target = x.sh->vals[1];
    in_bin = x.sh->vals[2];
    // red_* of this level stay untouched until after the next cluster barrier (start of the next level / gather)
    return bin;
}

constexpr int GATHER_CAP = MAX_TOPK;          // elements CTA 0 can sort
constexpr int GATHER_FAST = 1024;             // above this many elements in the crossing bin a second level pays off

// Selection inside `base`:
//   by_mass == false: the cut of the `need`-th largest element (1 <= need <= count inside base)
//   by_mass == true : the cut of the smallest ranking prefix whose mass reaches p * (mass inside base)
// Levels: a histogram of 2048 bins uniform in (M - y) whose width (a power of two) is chosen so that the bins just
// cover the row's finite range, and, if its crossing bin still holds more than GATHER_FAST elements, a second one
// that splits that bin 2048 ways; they spread any smooth logit distribution over many bins.  Then the elements of
// the crossing bin are gathered into CTA 0 and sorted.  Bins too crowded for that (massive ties) are
// resolved by three more levels over the key bits and an ordered tie count.
__device__ Cut select_cut(ExactCtx &x, const Cut &base, bool by_mass, unsigned long long need, float p,
                          unsigned long long *sortbuf) {
    unsigned long long target = need, in_bin = 0;
    const float Mf = x.Mf, scale = x.scale, inv_scale = x.inv_scale;
    auto dig_a = [=](uint32_t key) -> int {
        float t = fminf(__fmul_rn(__fsub_rn(Mf, unkey(key)), scale), 2047.0f);
        return 2047 - (int)t;
    };
    const int a = hist_level(x, base, by_mass, true, p, HBINS, dig_a, target, in_bin, sortbuf);
    // A bin is an interval of (M - y), hence of keys.  A conservative key interval (the exact one widened by a
    // margin that covers the roundings of the digit arithmetic and of this computation) lets the later passes
    // reject almost every element with two integer compares before the exact digit test.
    const bool band_ok = (Mf > -CUDART_INF_F) && (Mf < CUDART_INF_F);
    const float marg = fmaxf(fabsf(Mf), 2048.0f * inv_scale) * 9.5367431640625e-07f;   // 2^-20 of the larger magnitude
    auto key_band = [&](float d_lo, float d_hi, bool open_below, uint32_t &klo, uint32_t &khi) {   // M - y in [d_lo, d_hi)
        klo = 0u; khi = 0xFFFFFFFFu;
        if (!band_ok) return;
        khi = okey((Mf - d_lo) + marg);
        if (!open_below) klo = okey((Mf - d_hi) - marg);
    };
    uint32_t klo_a, khi_a;
    {
        const int n = 2047 - a;
        key_band((float)n * inv_scale, (float)(n + 1) * inv_scale, n == 2047, klo_a, khi_a);
    }
    auto dig_b = [=](uint32_t key) -> int {
        if (key < klo_a || key > khi_a) return -1;
        float t = __fmul_rn(__fsub_rn(Mf, unkey(key)), scale);
        int aa = (int)fminf(t, 2047.0f);
        if (2047 - aa != a) return -1;
        float f = fminf(__fmul_rn(__fsub_rn(t, (float)aa), 2048.0f), 2047.0f);
        return 2047 - (int)f;
    };
    // Smallest and largest key among the members of `base` that satisfy `inr` (one pass, one cluster barrier).
    // With low-precision logits a crowded bin is almost always ONE value repeated thousands of times; when the two
    // keys agree, the boundary value is known without further levels, gathering or sorting.
    auto value_span = [&](auto inr, uint32_t &gmin, uint32_t &gmax) {
        const uint32_t *keys = x.keys;
        const int len = x.len, lo_g = x.lo, per = x.per, tid = x.tid;
        const Cut bs = base;
        uint32_t kmn = 0xFFFFFFFFu, kmx = 0u;
        for (int i0 = 0; i0 < per; i0 += 4 * EX_THREADS) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * EX_THREADS + tid;
                if (i < len) {
                    const uint32_t key = keys[i];
                    if (member(bs, key, lo_g + i) && inr(key)) { kmn = min(kmn, key); kmx = max(kmx, key); }
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            kmx = max(kmx, __shfl_xor_sync(0xFFFFFFFFu, kmx, off));
            kmn = min(kmn, __shfl_xor_sync(0xFFFFFFFFu, kmn, off));
        }
        // one 64-bit word per warp carries both: the largest key and the complement of the smallest
        const unsigned long long both = ((unsigned long long)kmx << 32) | (uint32_t)(~kmn);
        __syncthreads();
        if (x.lane == 0) x.sh->wtot[x.warp] = both;
        __syncthreads();
        unsigned long long hi = 0, lo32 = 0;
        for (int w = 0; w < EX_WARPS; ++w) { hi = max(hi, x.sh->wtot[w] >> 32); lo32 = max(lo32, x.sh->wtot[w] & 0xFFFFFFFFull); }
        unsigned long long v[XV] = {hi, lo32, 0, 0};
        unsigned long long all[CL][XV];
        allgather(x, v, all);
        uint32_t gninv = 0;
        gmax = 0;
        for (int r = 0; r < CL; ++r) { gmax = max(gmax, (uint32_t)all[r][0]); gninv = max(gninv, (uint32_t)all[r][1]); }
        gmin = ~gninv;
    };
    bool single = false;                                          // the crossing bin holds one repeated value...
    uint32_t single_key = 0;                                      // ...this one
    int b = -1;
    if (in_bin > (unsigned long long)GATHER_FAST) {
        auto in_a = [=](uint32_t key) -> bool { return !(key < klo_a || key > khi_a) && dig_a(key) == a; };
        uint32_t gmin, gmax;
        value_span(in_a, gmin, gmax);
        if (gmin == gmax) { single = true; single_key = gmax; }
        else b = hist_level(x, base, by_mass, false, p, HBINS, dig_b, target, in_bin, sortbuf);
    }
    uint32_t klo = klo_a, khi = khi_a;
    if (b >= 0 && a != 0) {                                      // (bin 0 of level 0 is open below: no finer band)
        const int n = 2047 - a, m = 2047 - b;
        const float base_d = (float)n + (float)m * 0.00048828125f;              // aa + m / 2048, exact in fp32
        const float top_d = (m == 2047) ? (float)(n + 1) : base_d + 0.00048828125f;
        key_band(base_d * inv_scale, top_d * inv_scale, false, klo, khi);
    }
    auto in_range = [=](uint32_t key) -> bool {
        if (key < klo || key > khi) return false;
        if (dig_a(key) != a) return false;
        return b < 0 || dig_b(key) == b;
    };
    if (!single && in_bin <= (unsigned long long)GATHER_CAP) {
        // every CTA packs its elements of the bin into its own list, then the lists are laid end to end in
        // CTA 0, which sorts them and picks the element that completes the target
        if (x.tid == 0) x.sh->ucount = 0;
        __syncthreads();
        const uint32_t *keys = x.keys;
        const int len = x.len, lo_g = x.lo, per = x.per, tid = x.tid, lane = x.lane;
        unsigned int *ucount = &x.sh->ucount;
        const Cut bs = base;
        for (int i0 = 0; i0 < per; i0 += 4 * EX_THREADS) {
            uint32_t key[4];
            bool want[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * EX_THREADS + tid;
                key[u] = (i < len) ? keys[i] : 0u;
                want[u] = (i < len) && member(bs, key[u], lo_g + i) && in_range(key[u]);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * EX_THREADS + tid;
                const unsigned int pos = warp_append(ucount, want[u], lane);
                if (want[u] && pos < (unsigned int)GATHER_CAP) sortbuf[pos] = ((unsigned long long)key[u] << 32) | (uint32_t)(~(uint32_t)(lo_g + i));
            }
        }
        __syncthreads();
        const unsigned int mine = min(x.sh->ucount, (unsigned int)GATHER_CAP);
        unsigned long long v[XV] = {mine, 0, 0, 0};
        unsigned long long all[CL][XV];
        allgather(x, v, all);
        unsigned int off = 0, n = 0;
        for (int r = 0; r < CL; ++r) { if (r < x.rank) off += (unsigned int)all[r][0]; n += (unsigned int)all[r][0]; }
        if (x.rank != 0) {                      // CTA 0's own entries already sit at the front of its buffer
            unsigned long long *dst = cg::this_cluster().map_shared_rank(sortbuf, 0);
            for (unsigned int i = x.tid; i < mine; i += EX_THREADS)
                if (off + i < (unsigned int)GATHER_CAP) dst[off + i] = sortbuf[i];
        }
        cg::this_cluster().sync();
        unsigned long long v2[XV] = {0, 0, 0, 0};
        if (x.rank == 0) {
            const int nn = (int)min(n, (unsigned int)GATHER_CAP);
            const int m = next_pow2(nn);
            for (int i = nn + x.tid; i < m; i += EX_THREADS) sortbuf[i] = 0ull;
            __syncthreads();
            bitonic_sort_desc_cta<EX_THREADS>(sortbuf, m, x.tid);
            // running count / mass in ranking order; each thread owns a contiguous chunk of the sorted list
            const int chunk = (nn + EX_THREADS - 1) / EX_THREADS;
            const int lo = min(nn, x.tid * chunk), hi = min(nn, lo + chunk);
            unsigned long long mine = 0;
            for (int j = lo; j < hi; ++j) mine += by_mass ? qweight((uint32_t)(sortbuf[j] >> 32), Mf) : 1ull;
            // exclusive prefix over threads (warp scan, then warp totals)
            unsigned long long incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (x.lane >= o) incl += up;
            }
            __syncthreads();
            if (x.lane == 31) x.sh->wtot[x.warp] = incl;
            __syncthreads();
            unsigned long long woff = 0;
            for (int w = 0; w < x.warp; ++w) woff += x.sh->wtot[w];
            unsigned long long run = woff + incl - mine;
            if (x.tid == 0) x.sh->flag = nn - 1;
            __syncthreads();
            for (int j = lo; j < hi; ++j) {
                unsigned long long wj = by_mass ? qweight((uint32_t)(sortbuf[j] >> 32), Mf) : 1ull;
                if (run < target && run + wj >= target) x.sh->flag = j;
                run += wj;
            }
            __syncthreads();
            v2[0] = sortbuf[max(0, x.sh->flag)];
        }
        allgather(x, v2, all);
        Cut c;
        c.v = (uint32_t)(all[0][0] >> 32);
        c.idx = (int)(~(uint32_t)all[0][0]);
        return c;
    }
    // Crowded bin (or one repeated value, found above).  Once more the smallest and largest key in range are
    // compared (the range is narrower after a second level); if they still differ, the key bits of the elements in
    // range are descended, 11 + 11 + 10 at a time.
    uint32_t prefix = 0;
    int pbits = 0;
    if (!single) {
        uint32_t gmin, gmax;
        value_span(in_range, gmin, gmax);
        if (gmin == gmax) { single = true; single_key = gmax; }
    }
    if (single) { prefix = single_key; pbits = 32; }
    for (int pass = 0; pass < 3 && pbits < 32; ++pass) {
        const int nb = (pass < 2) ? 11 : 10;
        const int shift = 32 - pbits - nb;
        auto dig_k = [=](uint32_t key) -> int {
            if (pbits && (key >> (32 - pbits)) != prefix) return -1;
            if (!in_range(key)) return -1;
            return (int)((key >> shift) & ((1u << nb) - 1u));
        };
        const int d = hist_level(x, base, by_mass, false, p, 1 << nb, dig_k, target, in_bin, sortbuf);
        prefix = (prefix << nb) | (uint32_t)d;
        pbits += nb;
    }
    // prefix is the boundary value; `target` of its ties (by count) or enough of them to reach the mass
    unsigned long long r = target;
    if (by_mass) {
        unsigned long long qw = qweight(prefix, Mf);
        r = qw ? (target + qw - 1) / qw : 1;
    }
    if (r < 1) r = 1;
    if (r > in_bin) r = in_bin;
    const uint32_t v = prefix;
    const uint32_t *tkeys = x.keys;
    const int tlen = x.len, tlo = x.lo;
    const Cut tbase = base;
    auto tie = [=](int i) -> unsigned long long {
        return (i < tlen && tkeys[i] == v && member(tbase, v, tlo + i)) ? 1ull : 0ull;
    };
    OrderedState<unsigned long long> st;
    unsigned long long ntie, wdummy;
    ordered_totals<unsigned long long>(x, tie, tie, st, ntie);
    const int idx = ordered_find<unsigned long long>(x, r - 1, tie, st, wdummy);
    Cut c;
    c.v = v;
    c.idx = idx;
    return c;
}

// One row, start to finish, by the whole cluster.  Control flow is uniform over
// the cluster (every CTA executes the same sequence of cluster barriers).
template <int DT>
__device__ void exact_row(const KParams &P, const int row, ExactCtx &x, unsigned long long *sortbuf) {
    const RowCfg c = load_cfg(P, row);
    RowState *rs = P.rs + row;
    const int V = P.V;
    x.per = (((V + CL - 1) / CL) + 1023) & ~1023;
    x.lo = x.rank * x.per;
    x.len = max(0, min(V - x.lo, x.per));
    cg::this_cluster().sync();                               // every CTA of the cluster is resident before DSMEM traffic
    if (P.op == OP_VERIFY && c.l < P.K && P.draft_probs) {
        // verification rows read the draft distribution of their slice twice near the end of the row: ask for it now,
        // one 128-byte line per thread and trip, so that those reads find it in L2
        const float *q = P.draft_probs + ((size_t)c.b * P.K + c.l) * (size_t)V;
        for (int i = x.tid * 32; i < x.len; i += EX_THREADS * 32)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(q + x.lo + i));
    }

    // ---- load the slice, mask, sparse patches, temperature, keys
    constexpr int VEC = VecTraits<DT>::VEC;
    float *zf = reinterpret_cast<float *>(x.keys);
    const bool masked = (c.z & M_GRAMMAR) != 0;
    const uint32_t *mrow = masked ? P.bitmask + (long long)row * P.bitmask_stride : nullptr;
    const int nwords = (V + 31) >> 5;
#pragma unroll 4
    for (int li = x.tid * VEC; li < x.per; li += EX_THREADS * VEC) {
        const int first = x.lo + li;
        float vals[VEC];
        if (first < V) {
            uint4 raw;
            if (DT == 0) raw = __ldcs(reinterpret_cast<const uint4 *>(reinterpret_cast<const float *>(P.logits) + (long long)row * P.row_stride + first));
            else raw = __ldcs(reinterpret_cast<const uint4 *>(reinterpret_cast<const __nv_bfloat16 *>(P.logits) + (long long)row * P.row_stride + first));
            uint32_t r[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t mw = 0xFFFFFFFFu;
            if (masked) { int w = first >> 5; mw = (w < nwords ? __ldg(mrow + w) : 0u) >> (first & 31); }
#pragma unroll
            for (int q = 0; q < VEC; ++q) {
                float v;
                if (DT == 0) v = __uint_as_float(r[q]);
                else v = __uint_as_float((q & 1) ? (r[q >> 1] & 0xFFFF0000u) : (r[q >> 1] << 16));
                if (first + q >= V || !((mw >> q) & 1u)) v = -CUDART_INF_F;
                vals[q] = v;
            }
        } else {
#pragma unroll
            for (int q = 0; q < VEC; ++q) vals[q] = -CUDART_INF_F;
        }
#pragma unroll
        for (int q = 0; q < VEC; q += 4)
            *reinterpret_cast<float4 *>(zf + li + q) = make_float4(vals[q], vals[q + 1], vals[q + 2], vals[q + 3]);
    }
    __syncthreads();
    int bad = c.bad ? 1 : 0;
    if (c.hist_len > 0) {
        const int *hid = P.hist_ids + (long long)c.b * P.hist_stride;
        const int *hct = P.hist_counts + (long long)c.b * P.hist_stride;
        for (int t = x.tid; t < c.hist_len; t += EX_THREADS) {
            int id = __ldg(hid + t), ct = __ldg(hct + t);
            if (id < 0 || id >= V) { bad = 1; continue; }
            int li = id - x.lo;
            if (li >= 0 && li < x.len) zf[li] = apply_penalties(zf[li], ct, c);
        }
    }
    __syncthreads();
    if (c.bias_len > 0) {
        const int *bid = P.bias_ids + (long long)c.b * P.bias_stride;
        const float *bvl = P.bias_vals + (long long)c.b * P.bias_stride;
        for (int t = x.tid; t < c.bias_len; t += EX_THREADS) {
            int id = __ldg(bid + t);
            if (id < 0 || id >= V) { bad = 1; continue; }
            int li = id - x.lo;
            if (li >= 0 && li < x.len) zf[li] = __fadd_rn(zf[li], __ldg(bvl + t));
        }
    }
    bad = __syncthreads_or(bad);
    uint32_t kmax = 0, kmin = 0xFFFFFFFFu;      // kmin over the finite elements
    unsigned int nfin32 = 0;
    for (int l0 = x.tid * 4; l0 < x.per; l0 += EX_THREADS * 4) {   // per is a multiple of 1024: whole float4s
        const float4 z4 = *reinterpret_cast<const float4 *>(zf + l0);
        const float zz[4] = {z4.x, z4.y, z4.z, z4.w};
        uint32_t kk[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float y = c.temp ? div_tau(zz[u], c.tau) : zz[u];
            kk[u] = okey(y);
            kmax = max(kmax, kk[u]);
            const bool fin = (kk[u] > KEY_NEG_INF && l0 + u < x.len);
            nfin32 += fin ? 1u : 0u;
            if (fin) kmin = min(kmin, kk[u]);
        }
        *reinterpret_cast<uint4 *>(x.keys + l0) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
    }
    unsigned long long nfin = nfin32;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        kmax = max(kmax, __shfl_xor_sync(0xFFFFFFFFu, kmax, off));
        kmin = min(kmin, __shfl_xor_sync(0xFFFFFFFFu, kmin, off));
    }
    nfin = block_sum_u64(x, nfin);
    __syncthreads();
    if (x.lane == 0) { x.sh->wtot[x.warp] = kmax; x.sh->wcnt[x.warp] = kmin; }
    __syncthreads();
    for (int w = 0; w < EX_WARPS; ++w) { kmax = max(kmax, (uint32_t)x.sh->wtot[w]); kmin = min(kmin, (uint32_t)x.sh->wcnt[w]); }
    unsigned long long all[CL][XV];
    {
        unsigned long long v[XV] = {kmax, nfin, kmin, 0};
        allgather(x, v, all);
    }
    uint32_t Mkey = 0, mkey = 0xFFFFFFFFu;
    unsigned long long Nf = 0;
    for (int r = 0; r < CL; ++r) { Mkey = max(Mkey, (uint32_t)all[r][0]); Nf += all[r][1]; mkey = min(mkey, (uint32_t)all[r][2]); }
    x.Mf = unkey(Mkey);
    // Histogram resolution: 2048 bins uniform in (M - y) that just cover the row's finite range, the bin width a power
    // of two (so that scaling is exact); 32 bins per unit when the range is degenerate.
    {
        int e = 5;
        const float spread = (Nf > 0) ? __fsub_rn(x.Mf, unkey(mkey)) : 0.0f;
        if (spread > 0.0f && spread < CUDART_INF_F) e = max(-10, min(10, ilogbf(2040.0f / spread)));
        x.scale = ldexpf(1.0f, e);
        x.inv_scale = ldexpf(1.0f, -e);
    }
    const bool leader = (x.rank == 0 && x.tid == 0);

    if (__ldcg(&P.error[WS_ERROR]) & ERR_TIMEOUT) {           // (uniform over the cluster; see the merge kernel)
        if (leader && P.op != OP_TOPK) emit_row(P, c, row, -1, 0.0f, F_TIMEOUT | F_FALLBACK, 0, 0.0f);
        cg::this_cluster().sync();
        return;
    }
    if (bad) {
        if (leader) { emit_row(P, c, row, -1, 0.0f, F_BADPARAM | F_FALLBACK, 0, 0.0f); rs->status = 0; }
        cg::this_cluster().sync();
        return;
    }

    // ---------------------------------------------------------------- sonic_topk rows
    if (P.op == OP_TOPK) {
        Cut all_cut; all_cut.v = 0; all_cut.idx = -1;
        Cut cut = all_cut;
        if (c.k < V) cut = select_cut(x, all_cut, false, (unsigned long long)c.k, 1.0f, sortbuf);
        // compact the members into CTA 0's sort buffer
        if (x.tid == 0) x.sh->ucount = 0;
        __syncthreads();
        unsigned long long cnt = 0;
        for (int i = x.tid; i < x.len; i += EX_THREADS) cnt += member(cut, x.keys[i], x.lo + i) ? 1 : 0;
        cnt = block_sum_u64(x, cnt);
        unsigned long long v[XV] = {cnt, 0, 0, 0};
        allgather(x, v, all);
        unsigned int off = 0;
        for (int r = 0; r < x.rank; ++r) off += (unsigned int)all[r][0];
        unsigned long long *dst = cg::this_cluster().map_shared_rank(sortbuf, 0);
        for (int i0 = 0; i0 < x.len; i0 += EX_THREADS) {
            const int i = i0 + x.tid;
            const uint32_t key = (i < x.len) ? x.keys[i] : 0u;
            const bool want = (i < x.len) && member(cut, key, x.lo + i);
            const unsigned int pos = off + warp_append(&x.sh->ucount, want, x.lane);
            if (want && pos < (unsigned int)MAX_TOPK) dst[pos] = ((unsigned long long)key << 32) | (uint32_t)(~(uint32_t)(x.lo + i));
        }
        cg::this_cluster().sync();
        if (x.rank == 0) {
            const int n = min(c.k, MAX_TOPK);
            const int m = next_pow2(n);
            for (int i = n + x.tid; i < m; i += EX_THREADS) sortbuf[i] = 0ull;
            __syncthreads();
            bitonic_sort_desc_cta<EX_THREADS>(sortbuf, m, x.tid);
            for (int j = x.tid; j < n; j += EX_THREADS) {
                unsigned long long kv = sortbuf[j];
                P.out_vals[(size_t)row * P.ktop + j] = unkey((uint32_t)(kv >> 32));
                P.out_idx[(size_t)row * P.ktop + j] = (int)(~(uint32_t)kv);
            }
            if (x.tid == 0) rs->status = 0;
        }
        return;
    }

    // ---------------------------------------------------------------- sampling / verification rows
    if (Nf == 0) {
        if (leader) { emit_row(P, c, row, -1, 0.0f, F_NO_TOKEN | F_FALLBACK, 0, 0.0f); rs->status = 0; }
        cg::this_cluster().sync();
        return;
    }
    Cut cut; cut.v = KEY_NEG_INF; cut.idx = -1;            // every finite element
    if (c.k > 0 && (unsigned long long)c.k < Nf) cut = select_cut(x, cut, false, (unsigned long long)c.k, 1.0f, sortbuf);
    const Cut cut_k = cut;
    if (c.z & M_TOP_P) {
        Cut cp = select_cut(x, cut_k, true, 0ull, c.p, sortbuf);
        if (tighter(cp, cut)) cut = cp;
    }
    if (c.z & M_MIN_P) {
        double thr = (double)x.Mf + log((double)c.theta);
        float tf = (float)thr;
        if ((double)tf < thr) tf = nextafterf(tf, CUDART_INF_F);
        uint32_t tk = okey(tf);
        Cut cm; cm.v = tk - 1; cm.idx = -1;                // key >= tk
        if (tighter(cm, cut)) cut = cm;
    }
    // final support: size and mass in one ordered pass, then the draw in index order
    uint32_t a_acc, a_draw;
    draw_cells(P, c, a_acc, a_draw);
    // (the weight functions capture copies of what they read: a reference to the context would keep it in memory)
    const uint32_t *skeys = x.keys;
    const int slen = x.len, slo = x.lo;
    const float sMf = x.Mf;
    const Cut scut = cut;
    auto wq = [=](int i) -> unsigned long long {
        return (i < slen && member(scut, skeys[i], slo + i)) ? qweight(skeys[i], sMf) : 0ull;
    };
    auto inS = [=](int i) -> unsigned long long {
        return (i < slen && member(scut, skeys[i], slo + i)) ? 1ull : 0ull;
    };
    OrderedState<unsigned long long> stq;
    unsigned long long nS;
    ordered_totals<unsigned long long>(x, wq, inS, stq, nS);
    const unsigned long long Wq = stq.total;
    const unsigned long long mul = 2ull * a_draw + 1ull;               // u = mul / 2^25
    const unsigned long long T = (__umul64hi(Wq, mul) << 39) | ((Wq * mul) >> 25);
    // A position that carries a draft token needs a draw from p only if the draft is rejected AND the residual is
    // empty; every other row draws from p (below).
    const bool draft_pos = (P.op == OP_VERIFY && c.l < P.K);
    bool plain_draw = !draft_pos;
    int token = -1;

    uint32_t flags = F_FALLBACK;
    float p_draft = 0.0f;
    if (draft_pos) {
        const int d = P.draft_tokens[(size_t)c.b * P.K + c.l];
        const float *q = P.draft_probs + ((size_t)c.b * P.K + c.l) * (size_t)V;
        unsigned long long v[XV] = {0, 0, 0, 0};
        if (d >= x.lo && d < x.lo + x.len) v[0] = wq(d - x.lo) + 1ull;   // +1 marks the owner
        allgather(x, v, all);
        unsigned long long qd = 0;
        for (int r = 0; r < CL; ++r) if (all[r][0]) qd = all[r][0] - 1ull;
        double Pd = (double)qd / (double)Wq;
        double Q = (d >= 0 && d < V) ? (double)__ldg(q + d) : 0.0;
        const bool accept = (Pd > 0.0) && (cell_to_u(a_acc) * Q <= Pd);      // the same value in every CTA
        p_draft = (float)Pd;
        if (accept) {
            // the request moves on with the draft token: neither the residual nor a draw of this position is read
            flags |= F_ACCEPT;
            token = d;
        } else {
            // residual max(0, p - q) over the support, weights in fp64 (p - q cancels, so the weights must be accurate)
            const double Md = (double)x.Mf;
            auto wd = [=](int i) -> double {
                return (i < slen && member(scut, skeys[i], slo + i)) ? exp((double)unkey(skeys[i]) - Md) : 0.0;
            };
            OrderedState<double> std_;
            unsigned long long cdummy;
            ordered_totals<double>(x, wd, inS, std_, cdummy);
            const double Wd = std_.total;
            const double inv_Wd = 1.0 / Wd;                        // p = w * (1 / W): one rounding more than w / W, far below the margins
            auto rd = [=](int i) -> double {
                if (!(i < slen && member(scut, skeys[i], slo + i))) return 0.0;
                double r = exp((double)unkey(skeys[i]) - Md) * inv_Wd - (double)__ldg(q + slo + i);
                return r > 0.0 ? r : 0.0;
            };
            OrderedState<double> str;
            ordered_totals<double>(x, rd, inS, str, cdummy);
            if (str.total > 0.0) {
                double rw;
                token = ordered_find<double>(x, cell_to_u(a_draw) * str.total, rd, str, rw);
            }
            if (token < 0) {
                // empty residual (p <= q on the whole support, by rounding): draw from p itself; the ordered totals
                // of the fixed-point weights were overwritten by the passes above
                unsigned long long ndummy;
                ordered_totals<unsigned long long>(x, wq, inS, stq, ndummy);
                plain_draw = true;
            }
        }
    }
    double token_prob = 0.0;
    if (plain_draw) {
        unsigned long long qt = 0;
        token = ordered_find<unsigned long long>(x, T, wq, stq, qt);
        token_prob = (double)qt / (double)Wq;
    }
    if (leader) {
        emit_row(P, c, row, token, (float)token_prob, flags, (int)nS, p_draft);
        rs->status = 0;
    }
    cg::this_cluster().sync();
}

// Persistent clusters over the rows that need this path: the rows that are its own by class (top-k beyond what the
// streaming path sorts; the streaming kernel counts them) and the rows the streaming or histogram path could not
// finish (flagged and counted by their kernels).  The last kernel of a call's chain: it waits for its predecessor,
// puts the call's list counters back to zero and, in nearly every call, finds nothing to do and returns.
template <int DT>
__global__ void __cluster_dims__(CL, 1, 1) __launch_bounds__(EX_THREADS, 1)
sonic_exact_kernel(const KParams P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    ExactCtx x;
    x.rank = (int)cg::this_cluster().block_rank();
    x.tid = threadIdx.x; x.lane = x.tid & 31; x.warp = x.tid >> 5;
    x.phase = 0;
    x.keys = reinterpret_cast<uint32_t *>(smem_raw);
    x.hcnt = reinterpret_cast<unsigned int *>(smem_raw + SLICE_MAX * 4);
    x.hm0 = x.hcnt + HBINS; x.hm1 = x.hcnt + 2 * HBINS;
    x.sh = reinterpret_cast<ExactShared *>(smem_raw + SLICE_MAX * 4 + HBINS * 16);
    unsigned long long *sortbuf = reinterpret_cast<unsigned long long *>(smem_raw + SLICE_MAX * 4 + HBINS * 16 + 8192);
    uint32_t *need = reinterpret_cast<uint32_t *>(smem_raw + SLICE_MAX * 4 + HBINS * 16 + 8192 + MAX_TOPK * 8);

    KERNEL_T0(2);
    pdl_launch_dependents();
    pdl_wait_primary();
    const int ncl = gridDim.x / CL;
    const int cid = blockIdx.x / CL;
    const int nwords = (P.rows + 31) >> 5;
    // (the passes that read the two lists are complete: their lengths go back to zero for the next call)
    if (blockIdx.x == 0 && x.tid == 0) { P.error[WS_NDENSE] = 0u; P.error[WS_NRESID] = 0u; }
    if (__ldcg(&P.error[WS_ERROR]) & ERR_TIMEOUT) {
        // A bounded wait of the streaming kernel ran out (in this call or an earlier one on this workspace): nothing
        // the call computed is to be trusted.  This is the call's last kernel over the rows, behind both chains, so
        // here every row is made to say so (rows whose first tile was never processed are on no other path's list).
        for (int row = blockIdx.x * EX_THREADS + x.tid; row < P.rows; row += gridDim.x * EX_THREADS) {
            if (P.op == OP_TOPK) {
                for (int j = 0; j < P.ktop; ++j) { P.out_vals[(size_t)row * P.ktop + j] = -CUDART_INF_F; P.out_idx[(size_t)row * P.ktop + j] = -1; }
            } else {
                RowCfg c0;
                c0.b = row; c0.l = 0;
                emit_row(P, c0, row, -1, 0.0f, F_TIMEOUT, 0, 0.0f);
            }
        }
        KERNEL_T1(2);
        return;
    }
    // both counters stay as they are until the last cluster has left (below), so every CTA reads the same values
    if (__ldcg(&P.error[WS_FAILED_ROWS]) == 0u && __ldcg(&P.error[WS_NEXACT]) == 0u) { KERNEL_T1(2); return; }
    for (int i = x.tid; i < nwords; i += EX_THREADS) need[i] = 0u;
    __syncthreads();
    // every CTA marks the rows of the whole call (all derive the same list)
    for (int row = x.tid; row < P.rows; row += EX_THREADS) {
        const RowCfg c = load_cfg(P, row);
        const bool mine = (c.cls == CLS_EXACT) || (__ldcg(&P.rs[row].status) & ST_FAILED);
        if (mine) atomicOr(&need[row >> 5], 1u << (row & 31));
    }
    __syncthreads();
    int nmarked = 0;
    for (int w = 0; w < nwords; ++w) nmarked += __popc(need[w]);
    // The marked rows are handed out one at a time from a counter in the workspace header (rows differ a lot in
    // length); a cluster's first row needs no draw: the counter hands out ncl, ncl + 1, ...
    bool first = true;
    for (;;) {
        int t;
        if (first) {
            t = cid;
            first = false;
        } else {
            // the cluster's first thread draws the ordinal and leaves it in every CTA's shared memory
            if (x.rank == 0 && x.tid == 0) {
                const int drawn = ncl + (int)atomicAdd(&P.error[WS_EXACT_TICKET], 1u);
                for (int r = 0; r < CL; ++r) *cg::this_cluster().map_shared_rank(&x.sh->ticket, r) = drawn;
            }
            cg::this_cluster().sync();
            t = x.sh->ticket;                 // (the next write comes after the barriers of the row, or never)
        }
        if (t >= nmarked) break;
        int row = -1, seen = 0;
        for (int w = 0; w < nwords && row < 0; ++w) {
            const uint32_t bits = need[w];
            const int c = __popc(bits);
            if (t < seen + c) row = (w << 5) + (int)__fns(bits, 0, t - seen + 1);
            seen += c;
        }
        exact_row<DT>(P, row, x, sortbuf);
        KERNEL_T1(2);
    }
    // the last cluster to run out of rows puts the counters back to zero for the next call (every cluster has
    // drawn its final ordinal and read the row counts by then)
    if (x.rank == 0 && x.tid == 0) {
        const unsigned int left = atomicAdd(&P.error[WS_EXACT_LEFT], 1u);
        if (left == (unsigned int)(ncl - 1)) {
            P.error[WS_EXACT_TICKET] = 0u; P.error[WS_EXACT_LEFT] = 0u; P.error[WS_NEXACT] = 0u;
        }
    }
}

}  // namespace sonic
