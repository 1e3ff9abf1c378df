// Streaming kernel: reads every logit of the rows it owns exactly once, applies
// the logit-processing prologue, and reduces each 8192-element tile either to
// an argmax (greedy rows) or to the complete set of elements above a tile
// cutoff (top-k rows), written to the tile's own slot of the workspace without
// atomics.  The merge kernel (one CTA per row) then finishes the row: global
// top-k, truncation epilogue, token selection.  The two correspond to the
// paper's Algorithms "Stage 1: Tile-Local Reduction Kernel" and "Stage 2:
// Cross-Tile Merge and Selection Kernel"; the selection itself is ours.
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
template <> struct VecTraits<0> { static constexpr int VEC = 4, NV = 8; };
template <> struct VecTraits<1> { static constexpr int VEC = 8, NV = 4; };

// Loads one warp tile (1024 elements from wbase) into registers as fp32 and
// applies the grammar mask.  Elements at or beyond V read as -inf.
template <int DT>
__device__ __forceinline__ void load_warp_tile(const KParams &P, const RowCfg &c, long long row, int wbase, int lane,
                                               float (&e)[EPL]) {
    constexpr int VEC = VecTraits<DT>::VEC, NV = VecTraits<DT>::NV;
    const int V = P.V;
    uint4 raw[NV];
    if (DT == 0) {
        const float *rowp = reinterpret_cast<const float *>(P.logits) + row * P.row_stride;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int first = wbase + j * 32 * VEC + lane * VEC;
            raw[j] = make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u);
            if (first < V) raw[j] = __ldcs(reinterpret_cast<const uint4 *>(rowp + first));
        }
    } else {
        const __nv_bfloat16 *rowp = reinterpret_cast<const __nv_bfloat16 *>(P.logits) + row * P.row_stride;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int first = wbase + j * 32 * VEC + lane * VEC;
            raw[j] = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
            if (first < V) raw[j] = __ldcs(reinterpret_cast<const uint4 *>(rowp + first));
        }
    }
    uint32_t mw[NV];
    const bool masked = (c.z & M_GRAMMAR) != 0;
    if (masked) {
        const uint32_t *mrow = P.bitmask + row * P.bitmask_stride;
        const int nwords = (V + 31) >> 5;
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            int first = wbase + j * 32 * VEC + lane * VEC;
            int w = first >> 5;
            uint32_t word = (w < nwords) ? __ldg(mrow + w) : 0u;
            mw[j] = word >> (first & 31);
        }
    }
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        int first = wbase + j * 32 * VEC + lane * VEC;
        uint32_t r[4] = {raw[j].x, raw[j].y, raw[j].z, raw[j].w};
#pragma unroll
        for (int q = 0; q < VEC; ++q) {
            float v;
            if (DT == 0) v = __uint_as_float(r[q]);
            else v = __uint_as_float((q & 1) ? (r[q >> 1] & 0xFFFF0000u) : (r[q >> 1] << 16));
            if (first + q >= V) v = -CUDART_INF_F;
            if (masked && !((mw[j] >> q) & 1u)) v = -CUDART_INF_F;
            e[j * VEC + q] = v;
        }
    }
}

// Element index of register slot s of a lane.
template <int DT>
__device__ __forceinline__ int slot_index(int wbase, int lane, int s) {
    constexpr int VEC = VecTraits<DT>::VEC;
    return wbase + (s / VEC) * 32 * VEC + lane * VEC + (s % VEC);
}

// Sparse penalties and biases: the CTA stages its tile in shared memory, every
// thread scans a share of the row's lists and patches the entries that fall
// into this tile, then the lanes read their elements back.
template <int DT>
__device__ __forceinline__ void patch_tile(const KParams &P, const RowCfg &c, int row_tile_base, float *tile,
                                           int warp, int lane, int tid, bool report_bad, RowState *rs,
                                           float (&e)[EPL]) {
    constexpr int VEC = VecTraits<DT>::VEC, NV = VecTraits<DT>::NV;
    const int V = P.V;
    // prefetch the first list entries while the logits are still in flight
    const int *hid = P.hist_ids + (long long)c.b * P.hist_stride;
    const int *hct = P.hist_counts + (long long)c.b * P.hist_stride;
    const int *bid = P.bias_ids + (long long)c.b * P.bias_stride;
    const float *bvl = P.bias_vals + (long long)c.b * P.bias_stride;
    int h_id0 = -1, h_ct0 = 0, h_id1 = -1, h_ct1 = 0, b_id0 = -1;
    float b_v0 = 0.0f;
    if (tid < c.hist_len) { h_id0 = __ldg(hid + tid); h_ct0 = __ldg(hct + tid); }
    if (tid + STREAM_THREADS < c.hist_len) { h_id1 = __ldg(hid + tid + STREAM_THREADS); h_ct1 = __ldg(hct + tid + STREAM_THREADS); }
    if (tid < c.bias_len) { b_id0 = __ldg(bid + tid); b_v0 = __ldg(bvl + tid); }

#pragma unroll
    for (int j = 0; j < NV; ++j) {
        float *dst = tile + warp * WARP_TILE + j * 32 * VEC + lane * VEC;
#pragma unroll
        for (int q = 0; q < VEC; q += 4)
            *reinterpret_cast<float4 *>(dst + q) = make_float4(e[j * VEC + q], e[j * VEC + q + 1], e[j * VEC + q + 2], e[j * VEC + q + 3]);
    }
    __syncthreads();
    bool bad = false;
    auto pen = [&](int id, int ct) {
        if (id < 0 || id >= V) { bad = true; return; }
        int li = id - row_tile_base;
        if (li >= 0 && li < CTA_TILE) tile[li] = apply_penalties(tile[li], ct, c);
    };
    if (tid < c.hist_len) pen(h_id0, h_ct0);
    if (tid + STREAM_THREADS < c.hist_len) pen(h_id1, h_ct1);
    for (int t = tid + 2 * STREAM_THREADS; t < c.hist_len; t += STREAM_THREADS) pen(__ldg(hid + t), __ldg(hct + t));
    __syncthreads();
    auto add = [&](int id, float v) {
        if (id < 0 || id >= V) { bad = true; return; }
        int li = id - row_tile_base;
        if (li >= 0 && li < CTA_TILE) tile[li] = __fadd_rn(tile[li], v);
    };
    if (tid < c.bias_len) add(b_id0, b_v0);
    for (int t = tid + STREAM_THREADS; t < c.bias_len; t += STREAM_THREADS) add(__ldg(bid + t), __ldg(bvl + t));
    if (bad && report_bad) atomicOr(&rs->status, ST_BADID);
    __syncthreads();
#pragma unroll
    for (int j = 0; j < NV; ++j) {
        const float *src = tile + warp * WARP_TILE + j * 32 * VEC + lane * VEC;
#pragma unroll
        for (int q = 0; q < VEC; q += 4) {
            float4 v = *reinterpret_cast<const float4 *>(src + q);
            e[j * VEC + q] = v.x; e[j * VEC + q + 1] = v.y; e[j * VEC + q + 2] = v.z; e[j * VEC + q + 3] = v.w;
        }
    }
}

struct MergeShared {
    int count;
    int tcnt[MAX_TILES + 1];                   // exclusive prefix of the tiles' candidate counts
    unsigned int tkey;
    int n_p, n_m, pick;
    int found;
    double scratch[STREAM_THREADS];
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

// Row merge for top-k class rows, run by the CTA that finished the row's last
// tile.  buf is MERGE_CAP 64-bit words of shared memory (the staging tile,
// free by then).  Returns false if the candidates cannot prove the row's answer.
__device__ bool merge_topk_row(const KParams &P, const RowCfg &c, int row, int tiles,
                               unsigned long long *buf, MergeShared &sh, int tid) {
    const int cap_t = (int)(CAND_CAP / (unsigned)tiles);
    const TileRec *rec = P.tiles + (size_t)row * MAX_TILES;
    // tile records: one thread per tile, then a serial prefix over at most 32 entries
    if (tid == 0) { sh.count = 0; sh.tkey = 0; sh.found = 0; }
    __syncthreads();
    if (tid < tiles) {
        const unsigned int cnt = __ldcg(&rec[tid].cnt);
        sh.tcnt[tid + 1] = (int)cnt;
        atomicMax(&sh.tkey, __ldcg(&rec[tid].tkey));
        if (cnt > (unsigned int)cap_t) sh.found = 1;     // a tile overflowed its slot
    }
    __syncthreads();
    if (sh.found) return false;
    if (tid == 0) {
        sh.tcnt[0] = 0;
        for (int t = 0; t < tiles; ++t) sh.tcnt[t + 1] += sh.tcnt[t];
    }
    __syncthreads();
    const unsigned int tkey = sh.tkey;
    const bool complete = (tkey == KEY_NEG_INF);
    const bool strict = c.temp && !complete;            // keys are compared after the temperature division
    const uint32_t tykey = c.temp ? okey(__fdiv_rn(unkey(tkey), c.tau)) : tkey;
    const int total = sh.tcnt[tiles];
    for (int j = tid; j < total; j += STREAM_THREADS) {
        int t = 0;
        while (sh.tcnt[t + 1] <= j) ++t;
        unsigned long long cd = __ldcg(P.cand + (size_t)row * CAND_CAP + (size_t)t * cap_t + (j - sh.tcnt[t]));
        uint32_t zk = (uint32_t)(cd >> 32);
        if (zk < tkey) continue;
        uint32_t yk = zk;
        if (c.temp) yk = okey(__fdiv_rn(unkey(zk), c.tau));
        if (strict && yk <= tykey) continue;
        int pos = atomicAdd(&sh.count, 1);
        if (pos < MERGE_CAP) buf[pos] = ((unsigned long long)yk << 32) | (uint32_t)cd;
    }
    __syncthreads();
    const int Pn = sh.count;
    if (Pn > MERGE_CAP) return false;
    int n;
    if (Pn >= c.k) n = c.k;
    else if (complete && P.op != OP_TOPK) n = Pn;
    else return false;
    const int m = next_pow2(Pn);
    for (int i = Pn + tid; i < m; i += STREAM_THREADS) buf[i] = 0ull;
    __syncthreads();
    bitonic_sort_desc<STREAM_THREADS>(buf, m, tid);

    if (P.op == OP_TOPK) {
        for (int j = tid; j < n; j += STREAM_THREADS) {
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
    // shared-memory layout after the sort (n <= KFAST_SAMPLE = MERGE_CAP / 4):
    //   buf[0, n)     sorted keys (value key << 32 | ~index)
    //   w             weights exp(y - M) in ranking order
    //   cs            cumulative sums (ranking order), later residual / CDF in index order
    //   ik            (~index << 32 | ranking position), sorted descending = index ascending
    double *w = reinterpret_cast<double *>(buf + KFAST_SAMPLE);
    double *cs = reinterpret_cast<double *>(buf + 2 * KFAST_SAMPLE);
    unsigned long long *ik = buf + 3 * KFAST_SAMPLE;
    const double M = (double)unkey((uint32_t)(buf[0] >> 32));
    for (int j = tid; j < n; j += STREAM_THREADS) {
        double y = (double)unkey((uint32_t)(buf[j] >> 32));
        double wj = exp(y - M);
        w[j] = wj; cs[j] = wj;
    }
    if (tid == 0) { sh.n_p = n; sh.n_m = n; sh.found = 0; sh.pick = -1; }
    __syncthreads();
    block_inclusive_scan<STREAM_THREADS>(cs, n, sh.scratch, tid);
    const double Z = cs[n - 1];
    if (c.z & M_TOP_P) {
        const double target = (double)c.p * Z;
        for (int j = tid; j < n; j += STREAM_THREADS)
            if (cs[j] >= target && (j == 0 || cs[j - 1] < target)) sh.n_p = j + 1;
    }
    if (c.z & M_MIN_P) {
        const double thr = M + log((double)c.theta);
        for (int j = tid; j < n; j += STREAM_THREADS) {
            bool in = (double)unkey((uint32_t)(buf[j] >> 32)) >= thr;
            bool prev_in = (j == 0) || ((double)unkey((uint32_t)(buf[j - 1] >> 32)) >= thr);
            if (!in && prev_in) sh.n_m = j;
        }
    }
    __syncthreads();
    n = min(n, min(sh.n_p, sh.n_m));
    const double W = cs[n - 1];
    __syncthreads();
    // survivors in vocabulary-index order
    const int m2 = next_pow2(n);
    for (int j = tid; j < m2; j += STREAM_THREADS)
        ik[j] = (j < n) ? ((buf[j] << 32) | (unsigned long long)j) : 0ull;
    __syncthreads();
    bitonic_sort_desc<STREAM_THREADS>(ik, m2, tid);

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
        __syncthreads();
        for (int j = tid; j < n; j += STREAM_THREADS)
            if ((int)(~(uint32_t)(ik[j] >> 32)) == d) sh.pick = j;
        __syncthreads();
        double Pd = 0.0;
        if (sh.pick >= 0) Pd = w[(uint32_t)ik[sh.pick]] / W;
        double Q = (d >= 0 && d < P.V) ? (double)__ldg(q + d) : 0.0;
        bool accept = (Pd > 0.0) && (cell_to_u(a_acc) * Q <= Pd);
        p_draft = (float)Pd;
        if (accept) flags |= F_ACCEPT;
        __syncthreads();
        // residual max(0, p - q) over the support, in index order
        for (int j = tid; j < n; j += STREAM_THREADS) {
            int idx = (int)(~(uint32_t)(ik[j] >> 32));
            double r = w[(uint32_t)ik[j]] / W - (double)__ldg(q + idx);
            cs[j] = r > 0.0 ? r : 0.0;
        }
        __syncthreads();
        block_inclusive_scan<STREAM_THREADS>(cs, n, sh.scratch, tid);
        use_residual = cs[n - 1] > 0.0;
        __syncthreads();
    }
    if (!use_residual) {
        for (int j = tid; j < n; j += STREAM_THREADS) cs[j] = w[(uint32_t)ik[j]];
        __syncthreads();
        block_inclusive_scan<STREAM_THREADS>(cs, n, sh.scratch, tid);
    }
    const double R = cs[n - 1];
    const double target = u_draw * R;
    if (tid == 0) sh.pick = n - 1;
    __syncthreads();
    for (int j = tid; j < n; j += STREAM_THREADS)
        if (cs[j] > target && (j == 0 || !(cs[j - 1] > target))) sh.pick = j;
    __syncthreads();
    if (tid == 0) {
        int j = sh.pick;
        int token = (int)(~(uint32_t)(ik[j] >> 32));
        float prob = (float)(w[(uint32_t)ik[j]] / W);
        emit_row(P, c, row, token, prob, flags, n, p_draft);
    }
    return true;
}

template <int DT>
__global__ void __launch_bounds__(STREAM_THREADS, 4)
sonic_stream_kernel(const KParams P) {
    __shared__ __align__(16) float s_tile[CTA_TILE];
    __shared__ float s_tw[STREAM_WARPS];
    __shared__ int s_wcnt[STREAM_WARPS];
    __shared__ unsigned long long s_best[STREAM_WARPS];
    __shared__ int s_last;
    __shared__ MergeShared s_merge;

    const int row = blockIdx.y;
    const int tile = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowCfg c = load_cfg(P, row);
    RowState *rs = P.rs + row;
    if (c.cls == CLS_EXACT) return;
    TileRec *rec = P.tiles + (size_t)row * MAX_TILES + tile;
    const int tile_base = tile * CTA_TILE;
    const int wbase = tile_base + warp * WARP_TILE;

    float e[EPL];
    load_warp_tile<DT>(P, c, row, wbase, lane, e);
    if (c.hist_len > 0 || c.bias_len > 0)
        patch_tile<DT>(P, c, tile_base, s_tile, warp, lane, tid, tile == 0, rs, e);
    if (c.div_all) {
#pragma unroll
        for (int s = 0; s < EPL; ++s) e[s] = __fdiv_rn(e[s], c.tau);
    }

    constexpr int VEC = VecTraits<DT>::VEC, NV = VecTraits<DT>::NV;
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
                for (int s = EPL - 1; s >= 0; --s)
                    if (e[s] == wm) best = slot_index<DT>(wbase, lane, s);   // slots ascend with s: the last write is the lowest
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) best = min(best, __shfl_xor_sync(0xFFFFFFFFu, best, off));
            key = ((unsigned long long)okey(wm) << 32) | (uint32_t)(~(uint32_t)best);
        }
        if (lane == 0) s_best[warp] = key;
        __syncthreads();
        if (tid == 0) {
            unsigned long long b = s_best[0];
#pragma unroll
            for (int w = 1; w < STREAM_WARPS; ++w) b = max(b, s_best[w]);
            rec->best = b;
        }
    } else {
    // tile cutoff: minimum over G groups of the group maximum, then the largest over the CTA's warp tiles
    float g;
    const int G = c.G;
    if (G == 0) {
        g = -CUDART_INF_F;
    } else {
        const int L = (G >= 32) ? 1 : (32 / G);           // lanes per group
        g = (G == 64) ? fminf(h0, h1) : lm;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            float o = __shfl_xor_sync(0xFFFFFFFFu, g, off);
            g = (off < L) ? fmaxf(g, o) : fminf(g, o);
        }
    }
    if (lane == 0) s_tw[warp] = g;
    __syncthreads();
    float t = s_tw[0];
#pragma unroll
    for (int w = 1; w < STREAM_WARPS; ++w) t = fmaxf(t, s_tw[w]);
    // every finite element >= t goes to the tile's candidate slot
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
        int o = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += o;
    }
    if (lane == 31) s_wcnt[warp] = incl;
    __syncthreads();
    int base = 0, total = 0;
#pragma unroll
    for (int w = 0; w < STREAM_WARPS; ++w) {
        if (w == warp) base = total;
        total += s_wcnt[w];
    }
    const int cap_t = (int)(CAND_CAP / gridDim.x);
    if (cnt > 0 && total <= cap_t) {
        unsigned long long *dst = P.cand + (size_t)row * CAND_CAP + (size_t)tile * cap_t + base + (incl - cnt);
#pragma unroll
        for (int j = 0; j < NV; ++j) {
            if (mv[j] >= t) {
#pragma unroll
                for (int q = 0; q < VEC; ++q) {
                    float v = e[j * VEC + q];
                    if (v >= t && v > -CUDART_INF_F) {
                        int idx = slot_index<DT>(wbase, lane, j * VEC + q);
                        *dst++ = ((unsigned long long)okey(v) << 32) | (uint32_t)(~(uint32_t)idx);
                    }
                }
            }
        }
    }
    if (tid == 0) { rec->cnt = (unsigned int)total; rec->tkey = okey(t); }
    }

    // ---- the CTA that finishes the row's last tile merges the row while others keep streaming
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        const unsigned int done = atomicAdd(&rs->ticket, 1u);
        s_last = (done == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const int tiles = gridDim.x;
    const TileRec *recs = P.tiles + (size_t)row * MAX_TILES;
    const unsigned int status = __ldcg(&rs->status);
    bool ok = true;
    if (c.bad || (status & ST_BADID)) {
        if (tid == 0) emit_row(P, c, row, -1, 0.0f, F_BADPARAM, 0, 0.0f);
    } else if (c.cls == CLS_GREEDY) {
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
                    int token = (int)(~(uint32_t)best);
                    uint32_t flags = 0;
                    float pd = 0.0f;
                    if (P.op == OP_VERIFY && c.l < P.K) {
                        bool acc = P.draft_tokens[(size_t)c.b * P.K + c.l] == token;
                        if (acc) { flags |= F_ACCEPT; pd = 1.0f; }
                    }
                    emit_row(P, c, row, token, 1.0f, flags, 1, pd);
                }
            }
        }
    } else {
        ok = merge_topk_row(P, c, row, tiles, reinterpret_cast<unsigned long long *>(s_tile), s_merge, tid);
    }
    __syncthreads();
    if (tid == 0) {
        rs->ticket = 0;
        rs->status = ok ? 0u : ST_FAILED;
    }
}

}  // namespace sonic

