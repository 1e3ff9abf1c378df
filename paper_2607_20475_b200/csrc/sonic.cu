// C ABI of the sonic library (see include/sonic.h): argument validation and
// kernel launches.  Nothing here allocates device memory or synchronises.
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/sonic.h"
#include "sonic_common.cuh"
#include "sonic_dense.cuh"
#include "sonic_stream.cuh"
#include "sonic_exact.cuh"

namespace sonic {

// Verification epilogue: the K+1 positions of a request were resolved
// independently (accept flag, correction token); this scans them in order.
__global__ void sonic_verify_combine_kernel(const KParams P, int B) {
    KERNEL_T0(5);
    KERNEL_T1(5);
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const int K = P.K;
    int *toks = P.out_tokens + (size_t)b * (K + 1);
    uint32_t flags = 0;
    int acc = 0;
    bool decided = false;
    for (int l = 0; l <= K; ++l) {
        const PosResult r = P.pr[(size_t)b * (K + 1) + l];
        toks[l] = -1;
        if (l < K && P.out_pdraft) P.out_pdraft[(size_t)b * K + l] = (r.flags & (F_BADPARAM | F_NO_TOKEN)) ? 0.0f : r.p;
        if (r.flags & F_BADPARAM) flags |= F_BADPARAM;
        if (r.flags & F_TIMEOUT) flags |= F_TIMEOUT;
        if (decided) continue;
        flags |= (r.flags & F_FALLBACK);
        if (r.flags & F_NO_TOKEN) { flags |= F_NO_TOKEN; decided = true; continue; }
        if (l < K && (r.flags & F_ACCEPT)) { toks[l] = P.draft_tokens[(size_t)b * K + l]; acc = l + 1; }
        else { toks[l] = r.token; decided = true; }
    }
    if (flags & (F_BADPARAM | F_TIMEOUT)) {
        for (int l = 0; l <= K; ++l) toks[l] = -1;
        acc = 0;
        flags &= ~F_NO_TOKEN;
    }
    P.out_accept[b] = acc;
    P.out_flags[b] = flags;
}

constexpr size_t WS_HEADER = WS_HEADER_WORDS * 4;
constexpr int MERGE_SMEM = MERGE_CAP * 8;
constexpr int STREAM_SMEM_F32 = VecTraits<0>::NSTAGE * CTA_TILE * 4 + (int)sizeof(StreamShared<0>);
constexpr int STREAM_SMEM_BF16 = VecTraits<1>::NSTAGE * CTA_TILE * 2 + CTA_TILE * 4 + (int)sizeof(StreamShared<1>);
constexpr int EXACT_CLUSTERS = 4;             // clusters of the cluster kernel (its rows are rare)
constexpr int EXACT_SMEM = SLICE_MAX * 4 + HBINS * 16 + 8192 + MAX_TOPK * 8 + 8192;
static_assert(MERGE_SMEM >= DENSE_DYN_SMEM, "stage 2 of the histogram path runs in the merge kernel's shared memory");
static_assert(DENSE_THREADS == MERGE_THREADS, "stage 2 of the histogram path runs in the merge kernel's CTAs");

static thread_local char g_err[256] = "";

static int fail(int code, const char *msg) {
    snprintf(g_err, sizeof(g_err), "%s", msg);
    return code;
}
static int fail_cuda(cudaError_t e, const char *what) {
    snprintf(g_err, sizeof(g_err), "%s: %s", what, cudaGetErrorString(e));
    return SONIC_ECUDA;
}

// Workspace layout.  Only the header (WS_HEADER bytes at offset 0) is shared by all calls and must be zero between
// them; everything behind it is laid out for the shape of the call at hand (rows, V, whether the histogram path
// can be taken) and initialised by the call's own kernels, so one workspace serves calls of any shape that fits.
struct Layout {
    size_t rs, pr, tiles, cand, drow, dtile, dlist, rlist, hist, members, ykeys, total;
    unsigned int cand_stride;
    int ytiles;
};
static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
// Candidate slots per row: CAND_CAP, twice that for sonic_topk with k beyond 2048 (its tiles bring up to ~1100
// candidates each at k = 4096, V = 2^18, where an even share of CAND_CAP is 1024), never more than the row has elements.
static size_t slot_cap(int op, int ktop) { return (op == OP_TOPK && ktop > 2048) ? 2 * (size_t)CAND_CAP : (size_t)CAND_CAP; }
static Layout layout_for(long long rows, int V, bool dense, size_t cap = CAND_CAP) {
    Layout L;
    memset(&L, 0, sizeof(L));
    const int tiles = (V + CTA_TILE - 1) / CTA_TILE;
    const size_t slots = (size_t)tiles * CTA_TILE < cap ? (size_t)tiles * CTA_TILE : cap;
    L.cand_stride = (unsigned int)slots;
    L.ytiles = tiles;
    size_t off = WS_HEADER;
    L.rs = off;    off = align256(off + (size_t)rows * sizeof(RowState));
    L.pr = off;    off = align256(off + (size_t)rows * sizeof(PosResult));
    L.tiles = off; off = align256(off + (size_t)rows * sizeof(TileRec) * MAX_TILES);
    L.cand = off;  off = align256(off + (size_t)rows * slots * 8);
    if (dense) {
        L.drow = off;    off = align256(off + (size_t)rows * sizeof(DenseRow));
        L.dtile = off;   off = align256(off + (size_t)rows * sizeof(DenseTile) * MAX_TILES);
        L.dlist = off;   off = align256(off + (size_t)rows * 4);
        L.rlist = off;   off = align256(off + (size_t)rows * 4);
        L.hist = off;    off = align256(off + (size_t)rows * DBINS * 8);
        L.members = off; off = align256(off + (size_t)rows * MEMBER_CAP * 8);
        L.ykeys = off;   off = align256(off + (size_t)rows * tiles * CTA_TILE * 4);
    }
    L.total = off;
    return L;
}

static int g_sm_count[64];

static int configure_once(int *sm_count, int *device) {
    static std::once_flag once[64];
    static cudaError_t result[64];
    static int clusters[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(SONIC_EINVAL, "device ordinal out of range");
    std::call_once(once[dev], [&] {
        cudaError_t r = cudaSuccess;
        auto set = [&](const void *f, int bytes) {
            if (r == cudaSuccess) r = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
        };
        set((const void *)sonic_merge_kernel, MERGE_SMEM);
        set((const void *)sonic_dense_collect_kernel, DENSE_DYN_SMEM);
        set((const void *)sonic_dense_stage2_kernel, DENSE_DYN_SMEM);
        set((const void *)sonic_dense_finish_kernel, DENSE_DYN_SMEM);
        set((const void *)sonic_stream_kernel<0>, STREAM_SMEM_F32);
        set((const void *)sonic_stream_kernel<1>, STREAM_SMEM_BF16);
        if (r == cudaSuccess) r = cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
        set((const void *)sonic_exact_kernel<0>, EXACT_SMEM);
        set((const void *)sonic_exact_kernel<1>, EXACT_SMEM);
        int n = 0;
        if (r == cudaSuccess) {
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3(CL * EXACT_CLUSTERS);
            cfg.blockDim = dim3(EX_THREADS);
            cfg.dynamicSmemBytes = EXACT_SMEM;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = CL; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            r = cudaOccupancyMaxActiveClusters(&n, (const void *)sonic_exact_kernel<0>, &cfg);
        }
        clusters[dev] = n;
        result[dev] = r;
    });
    if (result[dev] != cudaSuccess) return fail_cuda(result[dev], "kernel configuration");
    if (clusters[dev] < 1) return fail(SONIC_ECUDA, "no 8-CTA cluster of the cluster kernel fits on this device");
    *sm_count = g_sm_count[dev] > 0 ? g_sm_count[dev] : 1;
    *device = dev;
    return SONIC_OK;
}

// Per host thread and device: one internal stream and two events, so that the histogram passes (rows with top-k off)
// run beside the merges (rows with top-k) instead of behind them.  A call forks the stream from the caller's after
// the streaming kernel and joins it before the call's last kernel; under stream capture it is captured with the
// caller's stream.  Created by the thread's first call on a device outside a capture; whenever the stream cannot
// be used safely (not created yet and the caller is capturing; still part of another, open capture) the call runs all
// of its kernels on the caller's stream instead, with the same results.
struct SideStream {
    cudaStream_t s = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool tried = false, ok = false;
    ~SideStream() {
        if (join) cudaEventDestroy(join);
        if (fork) cudaEventDestroy(fork);
        if (s) cudaStreamDestroy(s);
    }
};
static thread_local SideStream g_side[64];

static SideStream *side_stream_for(int dev, cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone, ss = cudaStreamCaptureStatusNone;
    unsigned long long cid = 0, sid = 0;
    if (cudaStreamGetCaptureInfo(st, &cs, &cid) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (cs == cudaStreamCaptureStatusInvalidated) return nullptr;
    SideStream &S = g_side[dev];
    if (!S.tried) {
        if (cs != cudaStreamCaptureStatusNone) return nullptr;          // (nothing is created while a capture is open)
        S.tried = true;
        S.ok = cudaStreamCreateWithFlags(&S.s, cudaStreamNonBlocking) == cudaSuccess &&
               cudaEventCreateWithFlags(&S.fork, cudaEventDisableTiming) == cudaSuccess &&
               cudaEventCreateWithFlags(&S.join, cudaEventDisableTiming) == cudaSuccess;
        if (!S.ok) cudaGetLastError();
    }
    if (!S.ok) return nullptr;
    if (cudaStreamGetCaptureInfo(S.s, &ss, &sid) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (ss == cudaStreamCaptureStatusInvalidated) return nullptr;
    if (ss == cudaStreamCaptureStatusActive && !(cs == cudaStreamCaptureStatusActive && cid == sid)) return nullptr;   // busy in another capture
    return &S;
}

// One call = a chain of kernels on the caller's stream.  Up to the residual pass each is a programmatic dependent
// of the one before (it may begin launching while its predecessor runs; the paper overlaps its two stages the
// same way, Section 3.5):
//   stream kernel -> merge kernel (rows with top-k)
//                 \-> [histogram pass -> its row step -> collect pass -> its row step -> residual pass]   (rows with top-k off)
//   -> cluster kernel (an ordinary launch after all of it: rows no other path finished; usually none) -> [verification scan]
// The second line runs on the thread's internal stream beside the merges when that stream can be used, else behind
// them on the caller's stream.
static int launch_all(KParams &P, void *ws, size_t ws_bytes, cudaStream_t st, int B_requests) {
    if (!ws) return fail(SONIC_EINVAL, "workspace is NULL");
    if (((uintptr_t)ws & 255) != 0) return fail(SONIC_EINVAL, "workspace must be 256-byte aligned");
    const bool dense = (P.op != OP_TOPK);
    const Layout L = layout_for(P.rows, P.V, dense, slot_cap(P.op, P.ktop));
    if (ws_bytes < L.total) return fail(SONIC_EWORKSPACE, "workspace too small for this many rows of this vocabulary size");
    int sm_count = 1, dev = 0;
    int rc = configure_once(&sm_count, &dev);
    if (rc != SONIC_OK) return rc;
    unsigned char *base = reinterpret_cast<unsigned char *>(ws);
    P.error = reinterpret_cast<unsigned int *>(base);
    P.rs = reinterpret_cast<RowState *>(base + L.rs);
    P.pr = reinterpret_cast<PosResult *>(base + L.pr);
    P.tiles = reinterpret_cast<TileRec *>(base + L.tiles);
    P.cand = reinterpret_cast<unsigned long long *>(base + L.cand);
    P.cand_stride = L.cand_stride;
    P.ytiles = L.ytiles;
    if (dense) {
        P.drow = reinterpret_cast<DenseRow *>(base + L.drow);
        P.dtile = reinterpret_cast<DenseTile *>(base + L.dtile);
        P.dlist = reinterpret_cast<int *>(base + L.dlist);
        P.rlist = reinterpret_cast<int *>(base + L.rlist);
        P.hist = reinterpret_cast<unsigned long long *>(base + L.hist);
        P.members = reinterpret_cast<unsigned long long *>(base + L.members);
        P.ykeys = reinterpret_cast<unsigned int *>(base + L.ykeys);
    }

    const int tiles = (P.V + CTA_TILE - 1) / CTA_TILE;
    const long long nitems_ll = (long long)tiles * P.rows;
    if (nitems_ll > 0x7FFFFFFF) return fail(SONIC_ESHAPE, "rows x tiles too large");
    const int nitems = (int)nitems_ll;
    cudaError_t e;

    const int grid1 = nitems < sm_count * 3 ? nitems : sm_count * 3;       // persistent: three CTAs per SM
    // a CTA's first request to the work queue: seven eighths of an even share, at least one item
    int chunk = (int)((7ll * nitems) / (8ll * grid1));
    chunk = chunk < 1 ? 1 : chunk;
    const int cap_t = (int)(L.cand_stride / (unsigned)tiles);
    if (P.dtype == SONIC_DTYPE_F32) sonic_stream_kernel<0><<<grid1, STREAM_CTA_THREADS, STREAM_SMEM_F32, st>>>(P, tiles, nitems, chunk, cap_t);
    else sonic_stream_kernel<1><<<grid1, STREAM_CTA_THREADS, STREAM_SMEM_BF16, st>>>(P, tiles, nitems, chunk, cap_t);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail_cuda(e, "stream kernel launch");

    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.stream = st;
    cfg.attrs = &pdl;
    cfg.numAttrs = 1;
    // Fork: the histogram passes go to the thread's internal stream (if it can be used), behind the streaming
    // kernel and beside the merges.  After the fork every exit joins that stream again (also the failing ones: the
    // caller's stream, or its capture, must not be left with a branch that was never joined).
    SideStream *side = dense ? side_stream_for(dev, st) : nullptr;
    if (side) {
        if ((e = cudaEventRecord(side->fork, st)) != cudaSuccess) return fail_cuda(e, "cudaEventRecord");
        if ((e = cudaStreamWaitEvent(side->s, side->fork, 0)) != cudaSuccess) return fail_cuda(e, "cudaStreamWaitEvent");
    }
    auto unwind = [&](int code) {
        if (side && cudaEventRecord(side->join, side->s) == cudaSuccess) cudaStreamWaitEvent(st, side->join, 0);
        return code;
    };
    cfg.gridDim = dim3(P.rows);
    cfg.blockDim = dim3(MERGE_THREADS);
    cfg.dynamicSmemBytes = MERGE_SMEM;
    e = cudaLaunchKernelEx(&cfg, sonic_merge_kernel, P, tiles);
    if (e != cudaSuccess) return unwind(fail_cuda(e, "merge kernel launch"));
    if (dense) {
        // the passes of the histogram path take (row, tile part) items in a loop: two CTAs per SM at most (a tile is
        // cut into up to four parts when a call has few rows of that class: up to four CTAs per tile)
        const int dense_ctas = (int)(4ll * nitems < 2ll * sm_count ? 4ll * nitems : 2ll * sm_count);
        cudaLaunchConfig_t dcfg = cfg;
        dcfg.stream = side ? side->s : st;
        dcfg.gridDim = dim3(dense_ctas);
        dcfg.blockDim = dim3(DENSE_THREADS);
        dcfg.dynamicSmemBytes = DENSE_DYN_SMEM;
        cudaLaunchConfig_t fcfg = dcfg;              // row-level steps: one CTA per row of the call (rows of other classes leave at once)
        fcfg.gridDim = dim3(P.rows);
        // Stage 2 never waits for its predecessor in the stream.  On the internal stream it is an ordinary launch
        // behind the fork; on the caller's stream it is a programmatic dependent of the merge kernel, whose CTAs let
        // it go only after their own wait for the streaming kernel.
        cudaLaunchConfig_t d2cfg = dcfg;
        if (side) { d2cfg.attrs = nullptr; d2cfg.numAttrs = 0; }
        e = cudaLaunchKernelEx(&d2cfg, sonic_dense_stage2_kernel, P, tiles);
        if (e != cudaSuccess) return unwind(fail_cuda(e, "histogram pass launch"));
        e = cudaLaunchKernelEx(&dcfg, sonic_dense_collect_kernel, P, tiles);
        if (e != cudaSuccess) return unwind(fail_cuda(e, "collect pass launch"));
        e = cudaLaunchKernelEx(&fcfg, sonic_dense_finish_kernel, P, tiles);
        if (e != cudaSuccess) return unwind(fail_cuda(e, "row finish launch"));
        if (P.op == OP_VERIFY && P.K > 0) {
            dcfg.dynamicSmemBytes = 0;
            fcfg.dynamicSmemBytes = 0;
            e = cudaLaunchKernelEx(&dcfg, sonic_dense_resid_kernel, P, tiles);
            if (e != cudaSuccess) return unwind(fail_cuda(e, "residual pass launch"));
            e = cudaLaunchKernelEx(&fcfg, sonic_dense_resid_finish_kernel, P, tiles);
            if (e != cudaSuccess) return unwind(fail_cuda(e, "residual draw launch"));
        }
    }
    if (side) {
        if ((e = cudaEventRecord(side->join, side->s)) != cudaSuccess) return fail_cuda(e, "cudaEventRecord");
        if ((e = cudaStreamWaitEvent(st, side->join, 0)) != cudaSuccess) return fail_cuda(e, "cudaStreamWaitEvent");
    }
    // The cluster kernel is an ordinary launch: it starts when everything before it is complete (the merges as well
    // as the histogram passes, which ran beside them).
    const int clusters = P.rows < EXACT_CLUSTERS ? P.rows : EXACT_CLUSTERS;
    cfg.gridDim = dim3(clusters * CL);
    cfg.blockDim = dim3(EX_THREADS);
    cfg.dynamicSmemBytes = EXACT_SMEM;
    cfg.attrs = nullptr;
    cfg.numAttrs = 0;
    if (P.dtype == SONIC_DTYPE_F32) e = cudaLaunchKernelEx(&cfg, sonic_exact_kernel<0>, P);
    else e = cudaLaunchKernelEx(&cfg, sonic_exact_kernel<1>, P);
    if (e != cudaSuccess) return fail_cuda(e, "cluster kernel launch");
    if (P.op == OP_VERIFY) {
        sonic_verify_combine_kernel<<<(B_requests + 127) / 128, 128, 0, st>>>(P, B_requests);
        e = cudaGetLastError();
        if (e != cudaSuccess) return fail_cuda(e, "verify combine launch");
    }
    g_err[0] = 0;
    return SONIC_OK;
}

static int check_logits(const void *logits, int dtype, int rows, int V, long long row_stride) {
    if (!logits) return fail(SONIC_EINVAL, "logits is NULL");
    if (dtype != SONIC_DTYPE_F32 && dtype != SONIC_DTYPE_BF16) return fail(SONIC_ESHAPE, "dtype must be fp32 or bf16");
    if (rows < 1) return fail(SONIC_ESHAPE, "need at least one row");
    if (rows > 65535) return fail(SONIC_ESHAPE, "too many rows (65535 logit rows at most)");
    if (V < 1 || V > SONIC_MAX_VOCAB) return fail(SONIC_ESHAPE, "V outside 1..SONIC_MAX_VOCAB");
    const int vec = (dtype == SONIC_DTYPE_F32) ? 4 : 8;
    if (row_stride < V || row_stride % vec != 0) return fail(SONIC_ESHAPE, "row_stride must be >= V and a multiple of 16 bytes");
    if (((uintptr_t)logits & 15) != 0) return fail(SONIC_EINVAL, "logits must be 16-byte aligned");
    return SONIC_OK;
}

static int fill_sample(KParams &P, const sonic_sample_args *a, int rows) {
    if (!a->mode) return fail(SONIC_EINVAL, "mode is NULL");
    P.V = a->V;
    P.dtype = a->dtype;
    P.logits = a->logits;
    P.row_stride = a->row_stride;
    P.mode = a->mode;
    P.bitmask = a->bitmask;
    P.bitmask_stride = a->bitmask_stride;
    if (a->bitmask && a->bitmask_stride < (a->V + 31) / 32) return fail(SONIC_ESHAPE, "bitmask_stride below ceil(V/32)");
    P.temperature = a->temperature; P.top_k = a->top_k; P.top_p = a->top_p; P.min_p = a->min_p;
    P.rep = a->rep_penalty; P.freq = a->freq_penalty; P.pres = a->pres_penalty;
    P.hist_ids = a->hist_ids; P.hist_counts = a->hist_counts; P.hist_len = a->hist_len; P.hist_stride = a->hist_stride;
    P.bias_ids = a->bias_ids; P.bias_vals = a->bias_vals; P.bias_len = a->bias_len; P.bias_stride = a->bias_stride;
    P.seed = reinterpret_cast<const unsigned long long *>(a->seed);
    P.offset = reinterpret_cast<const unsigned long long *>(a->offset);
    P.rows = rows;
    return SONIC_OK;
}

}  // namespace sonic

using namespace sonic;

extern "C" {

size_t sonic_workspace_bytes(int max_rows, int max_vocab, int max_topk) {
    if (max_rows < 1) max_rows = 1;
    if (max_vocab < 1) max_vocab = 1;
    if (max_vocab > SONIC_MAX_VOCAB) max_vocab = SONIC_MAX_VOCAB;
    // the larger of the two layouts a call can have: sampling / verification (with the histogram path's regions), and
    // sonic_topk with its slots for max_topk
    const size_t a = layout_for(max_rows, max_vocab, true).total;
    const size_t b = layout_for(max_rows, max_vocab, false, slot_cap(OP_TOPK, max_topk)).total;
    return a > b ? a : b;
}

int sonic_workspace_init(void *workspace, size_t bytes, void *stream) {
    if (!workspace) return fail(SONIC_EINVAL, "workspace is NULL");
    if (((uintptr_t)workspace & 255) != 0) return fail(SONIC_EINVAL, "workspace must be 256-byte aligned");
    if (bytes < layout_for(1, 1, true).total) return fail(SONIC_EWORKSPACE, "workspace smaller than one row");
    cudaError_t e = cudaMemsetAsync(workspace, 0, WS_HEADER, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(e, "cudaMemsetAsync");
    // The calling thread's internal stream is created here already (if this is not inside a capture), so that a
    // thread whose very first sampling call is captured still gets the two-stream schedule.  Best effort: a call
    // that finds no usable internal stream runs on the caller's stream alone.
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) (void)side_stream_for(dev, (cudaStream_t)stream);
    else cudaGetLastError();
    g_err[0] = 0;
    return SONIC_OK;
}

int sonic_sample(const sonic_sample_args *a, void *workspace, size_t workspace_bytes, void *stream) {
    if (!a) return fail(SONIC_EINVAL, "args is NULL");
    if (a->struct_size != sizeof(sonic_sample_args)) return fail(SONIC_EINVAL, "sonic_sample_args.struct_size mismatch");
    int rc = check_logits(a->logits, a->dtype, a->B, a->V, a->row_stride);
    if (rc != SONIC_OK) return rc;
    if (!a->out_token || !a->out_prob || !a->out_flags) return fail(SONIC_EINVAL, "an output pointer is NULL");
    KParams P;
    memset(&P, 0, sizeof(P));
    P.op = OP_SAMPLE;
    rc = fill_sample(P, a, a->B);
    if (rc != SONIC_OK) return rc;
    P.out_token = a->out_token; P.out_prob = a->out_prob; P.out_flags = a->out_flags; P.out_support = a->out_support;
    return launch_all(P, workspace, workspace_bytes, (cudaStream_t)stream, a->B);
}

int sonic_verify(const sonic_verify_args *v, void *workspace, size_t workspace_bytes, void *stream) {
    if (!v) return fail(SONIC_EINVAL, "args is NULL");
    if (v->struct_size != sizeof(sonic_verify_args)) return fail(SONIC_EINVAL, "sonic_verify_args.struct_size mismatch");
    const sonic_sample_args *a = &v->s;
    if (a->struct_size != sizeof(sonic_sample_args)) return fail(SONIC_EINVAL, "sonic_sample_args.struct_size mismatch");
    if (v->K < 0 || v->K > 15) return fail(SONIC_ESHAPE, "K outside 0..15");
    if (a->B < 1 || a->B > 4095) return fail(SONIC_ESHAPE, "B outside 1..4095");
    const int rows = a->B * (v->K + 1);
    int rc = check_logits(a->logits, a->dtype, rows, a->V, a->row_stride);
    if (rc != SONIC_OK) return rc;
    if (!v->out_tokens || !v->out_accept_len || !a->out_flags) return fail(SONIC_EINVAL, "an output pointer is NULL");
    if (v->K > 0 && (!v->draft_tokens || !v->draft_probs)) return fail(SONIC_EINVAL, "draft_tokens / draft_probs is NULL");
    KParams P;
    memset(&P, 0, sizeof(P));
    P.op = OP_VERIFY;
    P.K = v->K;
    rc = fill_sample(P, a, rows);
    if (rc != SONIC_OK) return rc;
    P.draft_tokens = v->draft_tokens; P.draft_probs = v->draft_probs;
    P.out_tokens = v->out_tokens; P.out_accept = v->out_accept_len; P.out_pdraft = v->out_p_draft;
    P.out_flags = a->out_flags;
    return launch_all(P, workspace, workspace_bytes, (cudaStream_t)stream, a->B);
}

int sonic_topk(const void *logits, int dtype, int B, int V, int64_t row_stride, int k,
               float *out_vals, int32_t *out_idx, void *workspace, size_t workspace_bytes, void *stream) {
    int rc = check_logits(logits, dtype, B, V, row_stride);
    if (rc != SONIC_OK) return rc;
    if (k < 1 || k > V || k > SONIC_MAX_TOPK) return fail(SONIC_ESHAPE, "k outside 1..min(V, SONIC_MAX_TOPK)");
    if (!out_vals || !out_idx) return fail(SONIC_EINVAL, "an output pointer is NULL");
    KParams P;
    memset(&P, 0, sizeof(P));
    P.op = OP_TOPK;
    P.rows = B; P.V = V; P.dtype = dtype; P.logits = logits; P.row_stride = row_stride; P.ktop = k;
    P.out_vals = out_vals; P.out_idx = out_idx;
    return launch_all(P, workspace, workspace_bytes, (cudaStream_t)stream, B);
}

// ---------------------------------------------------------------- no-allocation variant
// Scratch of sonic_topk_static: a workspace for SONIC_STATIC_MAX_ROWS rows of the largest vocabulary that lives in
// the library image.  In host code this name is only a stand-in for the symbol; the device
// address the kernels need comes from cudaGetSymbolAddress (below), never from `&`.
constexpr size_t STATIC_WS_BYTES = WS_HEADER + 256 * 4 +
    (size_t)SONIC_STATIC_MAX_ROWS * (sizeof(RowState) + sizeof(PosResult) + sizeof(TileRec) * MAX_TILES + 2 * (size_t)CAND_CAP * 8);
static __device__ __align__(256) unsigned char g_static_workspace[STATIC_WS_BYTES];

static int static_workspace_address(void **out) {
    static std::once_flag once[64];
    static cudaError_t result[64];
    static void *address[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(SONIC_EINVAL, "device ordinal out of range");
    std::call_once(once[dev], [&] {          // once per device, with that device current
        void *p = nullptr;
        result[dev] = cudaGetSymbolAddress(&p, g_static_workspace);
        address[dev] = p;
    });
    if (result[dev] != cudaSuccess) return fail_cuda(result[dev], "cudaGetSymbolAddress");
    *out = address[dev];
    return SONIC_OK;
}

int sonic_topk_static(const void *logits, int dtype, int B, int V, int64_t row_stride, int k,
                      float *out_vals, int32_t *out_idx, void *stream) {
    int rc = check_logits(logits, dtype, B, V, row_stride);
    if (rc != SONIC_OK) return rc;
    if (B > SONIC_STATIC_MAX_ROWS) return fail(SONIC_ESHAPE, "sonic_topk_static handles at most SONIC_STATIC_MAX_ROWS rows per call");
    if (k < 1 || k > V || k > SONIC_MAX_TOPK) return fail(SONIC_ESHAPE, "k outside 1..min(V, SONIC_MAX_TOPK)");
    if (!out_vals || !out_idx) return fail(SONIC_EINVAL, "an output pointer is NULL");
    void *ws = nullptr;
    rc = static_workspace_address(&ws);
    if (rc != SONIC_OK) return rc;
    // the array keeps whatever the previous call left: the header's control words must start at zero
    cudaError_t e = cudaMemsetAsync(ws, 0, WS_HEADER, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(e, "cudaMemsetAsync");
    KParams P;
    memset(&P, 0, sizeof(P));
    P.op = OP_TOPK;
    P.rows = B; P.V = V; P.dtype = dtype; P.logits = logits; P.row_stride = row_stride; P.ktop = k;
    P.out_vals = out_vals; P.out_idx = out_idx;
    return launch_all(P, ws, STATIC_WS_BYTES, (cudaStream_t)stream, B);
}

const char *sonic_last_error(void) { return g_err; }

}  // extern "C"
