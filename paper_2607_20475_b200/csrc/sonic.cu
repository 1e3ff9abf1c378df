// C ABI of the sonic library (see include/sonic.h): argument validation and
// kernel launches.  Nothing here allocates device memory or synchronises.
#include <cstdio>
#include <cstring>
#include <mutex>

#include "../../include/sonic.h"
#include "sonic_common.cuh"
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
        if (decided) continue;
        flags |= (r.flags & F_FALLBACK);
        if (r.flags & F_NO_TOKEN) { flags |= F_NO_TOKEN; decided = true; continue; }
        if (l < K && (r.flags & F_ACCEPT)) { toks[l] = P.draft_tokens[(size_t)b * K + l]; acc = l + 1; }
        else { toks[l] = r.token; decided = true; }
    }
    if (flags & F_BADPARAM) {
        for (int l = 0; l <= K; ++l) toks[l] = -1;
        acc = 0;
        flags &= ~F_NO_TOKEN;
    }
    P.out_accept[b] = acc;
    P.out_flags[b] = flags;
}

constexpr size_t WS_HEADER = 256;
constexpr int MERGE_SMEM = MERGE_CAP * 8;
constexpr int STREAM_SMEM_F32 = VecTraits<0>::NSTAGE * CTA_TILE * 4 + (int)sizeof(StreamShared<0>);
constexpr int STREAM_SMEM_BF16 = VecTraits<1>::NSTAGE * CTA_TILE * 2 + CTA_TILE * 4 + (int)sizeof(StreamShared<1>);
constexpr int SECOND_ROUND_CLUSTERS = 4;      // clusters of the exact kernel's second launch (rows the merge kernel failed)
constexpr int EXACT_SMEM = SLICE_MAX * 4 + HBINS * 16 + 8192 + MAX_TOPK * 8 + 8192;

static thread_local char g_err[256] = "";

static int fail(int code, const char *msg) {
    snprintf(g_err, sizeof(g_err), "%s", msg);
    return code;
}
static int fail_cuda(cudaError_t e, const char *what) {
    snprintf(g_err, sizeof(g_err), "%s: %s", what, cudaGetErrorString(e));
    return SONIC_ECUDA;
}

constexpr size_t WS_ROW_CTRL = sizeof(RowState) + sizeof(PosResult) + sizeof(TileRec) * MAX_TILES;
constexpr size_t WS_ROW = WS_ROW_CTRL + (size_t)CAND_CAP * 8;

static size_t ws_bytes_for(int rows) { return WS_HEADER + (size_t)rows * WS_ROW; }

static int g_max_clusters[64];      // co-resident 8-CTA clusters of the exact kernel, per device
static int g_sm_count[64];
// Per device: a side stream and two events.  The exact kernel's first round (rows that are its own by class) is
// forked onto the side stream at the start of a call and joined at its end, so that it runs beside the
// streaming and merge kernels of the caller's stream.  One call at a time uses them (g_launch_mutex).
static cudaStream_t g_side[64];
static cudaEvent_t g_fork[64], g_join[64];
static std::mutex g_launch_mutex[64];

static int configure_once(int *max_clusters, int *sm_count, int *device) {
    static std::once_flag once[64];
    static cudaError_t result[64];
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
        set((const void *)sonic_stream_kernel<0>, STREAM_SMEM_F32);
        set((const void *)sonic_stream_kernel<1>, STREAM_SMEM_BF16);
        if (r == cudaSuccess) r = cudaDeviceGetAttribute(&g_sm_count[dev], cudaDevAttrMultiProcessorCount, dev);
        set((const void *)sonic_exact_kernel<0>, EXACT_SMEM);
        set((const void *)sonic_exact_kernel<1>, EXACT_SMEM);
        int n = 0;
        if (r == cudaSuccess) {
            cudaLaunchConfig_t cfg;
            memset(&cfg, 0, sizeof(cfg));
            cfg.gridDim = dim3(CL * 64);
            cfg.blockDim = dim3(EX_THREADS);
            cfg.dynamicSmemBytes = EXACT_SMEM;
            cudaLaunchAttribute attr;
            attr.id = cudaLaunchAttributeClusterDimension;
            attr.val.clusterDim.x = CL; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
            cfg.attrs = &attr;
            cfg.numAttrs = 1;
            r = cudaOccupancyMaxActiveClusters(&n, (const void *)sonic_exact_kernel<0>, &cfg);
        }
        g_max_clusters[dev] = n;
        result[dev] = r;
    });
    if (result[dev] != cudaSuccess) return fail_cuda(result[dev], "kernel configuration");
    if (g_max_clusters[dev] < 1) return fail(SONIC_ECUDA, "no 8-CTA cluster of the exact kernel fits on this device");
    *max_clusters = g_max_clusters[dev];
    *sm_count = g_sm_count[dev] > 0 ? g_sm_count[dev] : 1;
    *device = dev;
    return SONIC_OK;
}

// Creates the side stream and its events on first use (never for sonic_topk_static, which forks nothing).
static int ensure_side(int dev) {
    static std::once_flag once[64];
    static cudaError_t result[64];
    std::call_once(once[dev], [&] {
        cudaError_t r = cudaStreamCreateWithFlags(&g_side[dev], cudaStreamNonBlocking);
        if (r == cudaSuccess) r = cudaEventCreateWithFlags(&g_fork[dev], cudaEventDisableTiming);
        if (r == cudaSuccess) r = cudaEventCreateWithFlags(&g_join[dev], cudaEventDisableTiming);
        result[dev] = r;
    });
    if (result[dev] != cudaSuccess) return fail_cuda(result[dev], "side stream creation");
    return SONIC_OK;
}

static int launch_all(KParams &P, void *ws, size_t ws_bytes, cudaStream_t st, int B_requests, bool fork = true) {
    if (!ws) return fail(SONIC_EINVAL, "workspace is NULL");
    if (((uintptr_t)ws & 255) != 0) return fail(SONIC_EINVAL, "workspace must be 256-byte aligned");
    if (ws_bytes < ws_bytes_for(P.rows)) return fail(SONIC_EWORKSPACE, "workspace too small for this many rows");
    int max_clusters = 0, sm_count = 1, dev = 0;
    int rc = configure_once(&max_clusters, &sm_count, &dev);
    if (rc != SONIC_OK) return rc;
    // the layout depends on the row capacity the workspace was sized for, recovered from its size
    const size_t cap_rows = (ws_bytes - WS_HEADER) / WS_ROW;
    unsigned char *base = reinterpret_cast<unsigned char *>(ws);
    P.error = reinterpret_cast<unsigned int *>(base);
    P.rs = reinterpret_cast<RowState *>(base + WS_HEADER);
    P.pr = reinterpret_cast<PosResult *>(base + WS_HEADER + cap_rows * sizeof(RowState));
    P.tiles = reinterpret_cast<TileRec *>(base + WS_HEADER + cap_rows * (sizeof(RowState) + sizeof(PosResult)));
    P.cand = reinterpret_cast<unsigned long long *>(base + WS_HEADER + cap_rows * WS_ROW_CTRL);

    const int tiles = (P.V + CTA_TILE - 1) / CTA_TILE;
    const long long nitems_ll = (long long)tiles * P.rows;
    if (nitems_ll > 0x7FFFFFFF) return fail(SONIC_ESHAPE, "rows x tiles too large");
    const int nitems = (int)nitems_ll;
    std::lock_guard<std::mutex> lock(g_launch_mutex[dev]);
    cudaError_t e;

    // Fork: the exact kernel's first round goes to the side stream BEFORE the streaming kernel is launched, so that
    // its clusters (one SM per CTA) are placed first; clusters without a row leave at once and the streaming
    // kernel's CTAs, which take their tiles from a queue, fill whatever is free.  Without the fork (the entry
    // point that creates no resources) both rounds run in one launch after the merge kernel.
    cudaLaunchConfig_t xcfg;
    memset(&xcfg, 0, sizeof(xcfg));
    xcfg.gridDim = dim3((P.rows < max_clusters ? P.rows : max_clusters) * CL);
    xcfg.blockDim = dim3(EX_THREADS);
    xcfg.dynamicSmemBytes = EXACT_SMEM;
    if (fork) {
        rc = ensure_side(dev);
        if (rc != SONIC_OK) return rc;
        xcfg.stream = g_side[dev];
        if ((e = cudaEventRecord(g_fork[dev], st)) != cudaSuccess) return fail_cuda(e, "cudaEventRecord");
        if ((e = cudaStreamWaitEvent(g_side[dev], g_fork[dev], 0)) != cudaSuccess) return fail_cuda(e, "cudaStreamWaitEvent");
        if (P.dtype == SONIC_DTYPE_F32) e = cudaLaunchKernelEx(&xcfg, sonic_exact_kernel<0>, P, 1);
        else e = cudaLaunchKernelEx(&xcfg, sonic_exact_kernel<1>, P, 1);
        if (e != cudaSuccess) return fail_cuda(e, "exact kernel launch (first round)");
        if ((e = cudaEventRecord(g_join[dev], g_side[dev])) != cudaSuccess) return fail_cuda(e, "cudaEventRecord");
    }

    // after the fork every exit joins the side stream again (also the failing ones: the caller's stream, or its
    // capture, must not be left with a branch that was never joined)
    auto unwind = [&](int code) {
        if (fork) cudaStreamWaitEvent(st, g_join[dev], 0);
        return code;
    };
    const int grid1 = nitems < sm_count * 3 ? nitems : sm_count * 3;       // persistent: three CTAs per SM
    // a CTA's first request to the work queue: seven eighths of an even share, at least one item
    int chunk = (int)((7ll * nitems) / (8ll * grid1));
    chunk = chunk < 1 ? 1 : chunk;
    if (P.dtype == SONIC_DTYPE_F32) sonic_stream_kernel<0><<<grid1, STREAM_CTA_THREADS, STREAM_SMEM_F32, st>>>(P, tiles, nitems, chunk, (int)(CAND_CAP / (unsigned)tiles));
    else sonic_stream_kernel<1><<<grid1, STREAM_CTA_THREADS, STREAM_SMEM_BF16, st>>>(P, tiles, nitems, chunk, (int)(CAND_CAP / (unsigned)tiles));
    e = cudaGetLastError();
    if (e != cudaSuccess) return unwind(fail_cuda(e, "stream kernel launch"));
    // the merge kernel and the exact kernel's second round are programmatic dependents: they may begin launching
    // while their predecessor still runs and synchronise on it inside the kernel
    cudaLaunchAttribute pdl;
    pdl.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl.val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.stream = st;
    cfg.attrs = &pdl;
    cfg.numAttrs = 1;
    cfg.gridDim = dim3(P.rows);
    cfg.blockDim = dim3(MERGE_THREADS);
    cfg.dynamicSmemBytes = MERGE_SMEM;
    e = cudaLaunchKernelEx(&cfg, sonic_merge_kernel, P, tiles);
    if (e != cudaSuccess) return unwind(fail_cuda(e, "merge kernel launch"));

    // rows the merge kernel cannot prove are rare: a few clusters suffice for the second round (the full set when
    // this launch also runs the first round)
    const int clusters2 = fork ? (P.rows < SECOND_ROUND_CLUSTERS ? P.rows : (max_clusters < SECOND_ROUND_CLUSTERS ? max_clusters : SECOND_ROUND_CLUSTERS))
                               : (P.rows < max_clusters ? P.rows : max_clusters);
    cfg.gridDim = dim3(clusters2 * CL);
    cfg.blockDim = dim3(EX_THREADS);
    cfg.dynamicSmemBytes = EXACT_SMEM;
    const int rounds = fork ? 2 : 3;
    if (P.dtype == SONIC_DTYPE_F32) e = cudaLaunchKernelEx(&cfg, sonic_exact_kernel<0>, P, rounds);
    else e = cudaLaunchKernelEx(&cfg, sonic_exact_kernel<1>, P, rounds);
    if (e != cudaSuccess) return unwind(fail_cuda(e, "exact kernel launch (second round)"));

    // join: everything after this call in the caller's stream sees the first round's rows too
    if (fork && (e = cudaStreamWaitEvent(st, g_join[dev], 0)) != cudaSuccess) return fail_cuda(e, "cudaStreamWaitEvent");
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

size_t sonic_workspace_bytes(int max_rows) {
    if (max_rows < 1) max_rows = 1;
    return ws_bytes_for(max_rows);
}

int sonic_workspace_init(void *workspace, size_t bytes, void *stream) {
    if (!workspace) return fail(SONIC_EINVAL, "workspace is NULL");
    if (bytes < ws_bytes_for(1)) return fail(SONIC_EWORKSPACE, "workspace smaller than one row");
    const size_t cap_rows = (bytes - WS_HEADER) / WS_ROW;
    cudaError_t e = cudaMemsetAsync(workspace, 0, WS_HEADER + cap_rows * WS_ROW_CTRL, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(e, "cudaMemsetAsync");
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
// Scratch of sonic_topk_static: a workspace for SONIC_STATIC_MAX_ROWS rows that lives in
// the library image.  In host code this name is only a stand-in for the symbol; the device
// address the kernels need comes from cudaGetSymbolAddress (below), never from `&`.
static __device__ __align__(256) unsigned char g_static_workspace[WS_HEADER + (size_t)SONIC_STATIC_MAX_ROWS * WS_ROW];

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
    const size_t bytes = WS_HEADER + (size_t)SONIC_STATIC_MAX_ROWS * WS_ROW;
    // the array keeps whatever the previous call left: the control words must start at zero
    cudaError_t e = cudaMemsetAsync(ws, 0, WS_HEADER + (size_t)SONIC_STATIC_MAX_ROWS * WS_ROW_CTRL, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail_cuda(e, "cudaMemsetAsync");
    KParams P;
    memset(&P, 0, sizeof(P));
    P.op = OP_TOPK;
    P.rows = B; P.V = V; P.dtype = dtype; P.logits = logits; P.row_stride = row_stride; P.ktop = k;
    P.out_vals = out_vals; P.out_idx = out_idx;
    return launch_all(P, ws, bytes, (cudaStream_t)stream, B, /*fork=*/false);     // creates no stream or event either
}

const char *sonic_last_error(void) { return g_err; }

}  // extern "C"
