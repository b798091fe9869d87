// Host side of the C ABI declared in include/psgd.h: argument checks, workspace
// layout and the stream-ordered sequence of kernels for one iteration of
// Algorithm 2 (SSP-Comp or SVD-Comp of Algorithm 1 plus the residual update).
#include "../../include/psgd.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <utility>
#include <vector>

#include "psgd_kernels.cuh"
#include "psgd_fused.cuh"
#include "psgd_gemm_tc.cuh"
#include "psgd_stream.cuh"
#include "psgd_backproject_tma.cuh"

using namespace psgd;

namespace {

constexpr int MAX_R = 128;
constexpr int MAX_L = 160;  // widest refresh block
constexpr int PENDING_TC_MIN_R = 8;    // above this many columns the pending-residual projection runs on the tensor cores by default
constexpr int REFRESH_F32_TAIL = 4;   // float32-accurate sweeps that end a refresh whose early sweeps ran in TF32

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

struct Layout {
    size_t flags, defic, Pnode, Pmean, Phat, Qnode, part, gram, T, dbar, Y, Z, V, U, total;
    size_t Qpad, Ppad, Qsub, Tacc, Pout, Wpart, Cmat, Cpart;  // deferred (single-pass) mode only
    size_t dbarT, Yt, Zt, gpart;                              // tensor-core refresh only
    size_t rtP, rtQ;                                          // tensor-core residual (r > 16) only
    size_t Pold, dpart;                                       // stopping test of the refresh
    size_t ptQ;                                               // tensor-core projection: split transposed Q
    size_t ppP, ppQ;                                          // ... of the two-pass deferred mode: images of P~_prev and Qsub
    size_t sPpart, sCnt, sGram;                               // L2-pipelined single-pass kernel: per-unit partial products, counters and flags, Gram partials
};

struct ProfEvent {
    cudaEvent_t a, b;
    int kind;
};

// An encoded TMA descriptor together with everything it was encoded from.
struct CachedMap {
    const void* base;
    int64_t n, m, mats;
    int bw, rows, swizzle, bf16;
    CUtensorMap map;
};

}  // namespace

struct psgd_handle {
    int64_t m, n;
    int r, N, count, tau;
    uint64_t seed;
    int error_form = 0, mode = 0, refresh_iters = 0 /* 0: chosen from the block width */, refresh_warm = 1, oversample = -1, refresh_tc = 1, power_steps = 1, refresh_adaptive = 1;
    bool tc_ok = false;           // the refresh block is wide enough for the tensor-core sweeps
    size_t gpart_floats = 0;
    bool grad_bf16 = false;       // G arrives as bfloat16
    bool ptc_ok = false;          // projections of more than 16 columns on the tensor cores
    bool ppt_ok = false;          // pending-residual projection (two-pass deferred mode) on the tensor cores
    int pend_tc = 0;              // PSGD_OPT_PENDING_TC: 0 where it is the faster form, 1 wherever it fits, 2 never
    int ptc_ncp = 0;
    bool rtc_ok = false;          // ranks above 16 with 16-byte row strides: residual update on the tensor cores
    int rtc_KP = 0;
    int64_t t = 0;
    float* E = nullptr;
    float* Q = nullptr;
    char* ws = nullptr;
    size_t ws_bytes = 0;
    Layout lay{};
    int ell = 0;        // refresh block width
    int S = 1, rpc = 0; // back-projection row chunks
    int64_t launches = 0;
    bool profiling = false;
    std::vector<ProfEvent> events;
    std::vector<CachedMap> maps;  // tensor maps already encoded for this handle (E and the workspace never move after psgd_attach)
    size_t map_next = 0;          // slot the next new map replaces once the cache is full
    char err[256] = "no error";
    bool vec4 = false;  // n % 4 == 0 (128-bit paths usable when pointers are 16-byte aligned)
    // single-pass (deferred residual) plan and state
    bool fused_ok = false;        // the shape fits the cluster kernel
    int RP = 0, CS = 1, WC = 0, KC = 1, KCmax = 1, nblk = 0;
    size_t fused_smem = 0;
    int active_clusters = -1;     // clusters of the single-pass kernel resident at once (known after its first launch)
    bool pending = false;         // E holds Delta_t; the residual is Delta_t - P~_t Qsub^T
    bool pending_fused = false;   // ... and the padded factors the single-pass kernel subtracts are those of that step
    bool tacc_identity = true;    // no preconditioner yet
    bool qpad_valid = false;      // padded copy of Q is current
    // L2-pipelined single-pass kernel (psgd_stream.cuh)
    int single_pass_kernel = 0;   // PSGD_OPT_SINGLE_PASS: 0 the fastest known for the shape, 1 cluster kernel, 2 two-pass kernels, 3 L2-pipelined kernel
    bool stream_ok = false;       // the shape fits the L2-pipelined kernel
    int s_nrb = 0, s_ngrp = 0, s_tpu = 0, s_csplit = 0, s_KC = 1, s_CB = 0, s_grid = -1;
    bool transposed = false;      // PSGD_OPT_TRANSPOSED: G and E are stored as [n][m] (the transpose of the m x n problem)
    int t_S = 1, t_rpc = 0;       // row chunks of the contraction over the n stored rows (transposed storage)
    int step_kernel = 0;          // what ran the last step: 0 three-/two-pass kernels, 1 cluster kernel, 2 L2-pipelined kernel
    bool bq_ok = true;            // back-projection with TMA-staged tiles where the shape allows (PSGD_OPT_BACKPROJECT_TMA)
    bool ran_pending_tc = false;  // the projection of the step in flight folded the pending residual in on the tensor cores
    int ex_phase = 0;             // psgd_exchange_*: 0 between steps, 1 after _begin, 2 after _orth
    bool ex_refresh = false;      // the step in flight is a refresh
    int sm_count = 0;             // multiprocessors of the device that was current when the handle was created
};

namespace {

// Multiprocessors of the current device; 148 (a B200) when no device is visible, so that a handle can still be
// created and sized on a machine without one.
int device_sms() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
        return sms;
    cudaGetLastError();
    return 148;
}

// K splits of the tensor-core product with M rows and K columns: enough CTAs for about two per SM,
// at least 8 K-blocks of 32 each
int gemm_tc_splits(int64_t M, int64_t K, int count, int sms) {
    int64_t tiles = ((M + TC_BM - 1) / TC_BM) * count;
    int64_t KB = (K + TC_BK - 1) / TC_BK;
    int64_t S = std::max<int64_t>(1, std::min<int64_t>((2 * sms + tiles - 1) / tiles, std::max<int64_t>(1, KB / 8)));
    int64_t kbps = (KB + S - 1) / S;
    return (int)((KB + kbps - 1) / kbps);
}

int refresh_width(const psgd_handle* h) {
    int over = h->oversample >= 0 ? h->oversample : std::max(8, h->r);
    int ell = std::min<int64_t>(h->n, (int64_t)h->r + over);
    ell = std::min(ell, MAX_L);
    return std::max(ell, h->r);
}

void plan(psgd_handle* h) {
    h->ell = refresh_width(h);
    const int colblk = ceil_div(h->n, BP_COLS);
    const int64_t target = 8 * (int64_t)h->sm_count;
    int64_t base = (int64_t)h->count * h->N * colblk;
    int S = (int)std::max<int64_t>(1, (target + base - 1) / base);
    S = std::min<int64_t>(S, ceil_div(h->m, BP_SUB));
    int rpc = (int)align_up(ceil_div(h->m, S), BP_SUB);
    h->rpc = rpc;
    h->S = ceil_div(h->m, rpc);
    // refresh back-projection (Z = Dbar^T Y, one "node"): its own chunking, computed at launch,
    // but it shares the partial buffer, so size that for the larger of the two uses.
    Layout& L = h->lay;
    const size_t m = h->m, n = h->n, r = h->r, N = h->N, cnt = h->count, ell = h->ell;
    const size_t c = std::max<size_t>(r, ell);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.flags = take(256);
    L.defic = take(cnt * 192 * 4);
    L.Pnode = take(cnt * N * m * r * 4);
    L.Pmean = take(cnt * m * r * 4);
    L.Phat = take(cnt * m * r * 4);
    L.Qnode = take(cnt * N * n * r * 4);
    size_t part_step = cnt * N * (size_t)h->S * n * r * 4;
    size_t part_ref = cnt * (size_t)ceil_div(h->m, BP_SUB) * n * ell * 4;  // upper bound on chunks
    part_ref = std::min(part_ref, cnt * (size_t)64 * n * ell * 4);          // refresh uses <= 64 chunks
    if (h->transposed) {   // P_i = S_i^T Q contracts over the n stored rows and has m outputs per column of Q
        const int colblk_t = ceil_div(h->m, BP_COLS);
        int St = (int)std::max<int64_t>(1, (target + (int64_t)h->count * h->N * colblk_t - 1) / ((int64_t)h->count * h->N * colblk_t));
        St = std::min<int64_t>(St, ceil_div(h->n, BP_SUB));
        h->t_rpc = (int)align_up(ceil_div(h->n, St), BP_SUB);
        h->t_S = ceil_div(h->n, h->t_rpc);
        part_step = std::max(part_step, cnt * N * (size_t)h->t_S * m * r * 4);
    }
    L.part = take(std::max(part_step, part_ref));
    size_t nparts = std::max<size_t>(ceil_div(std::max(m, n), GR_ROWS), 64);  // 64: most clusters per matrix
    L.gram = take(cnt * nparts * c * c * 8);
    L.T = take(cnt * c * c * 8);
    L.dbar = take(cnt * m * n * 4);
    L.Y = take(cnt * m * ell * 4);
    L.Z = take(cnt * n * ell * 4);
    size_t c2 = (c + 1) & ~(size_t)1;
    L.V = take(std::max<size_t>(8, cnt * jac_log_doubles((int)c2) * 8));   // rotation log of the Rayleigh-Ritz step (blocks too wide for shared memory)
    L.U = take(cnt * ell * r * 8);
    L.Pold = take(cnt * m * r * 4);
    L.dpart = take(cnt * ((size_t)ceil_div(h->m, 64) + 1) * 8);
    // ---- tensor-core sweeps of the refresh: block of >= 8 columns, 16-byte row strides for TMA ----
    h->tc_ok = h->refresh_tc && ell >= 8 && ell <= TC_MAXN && h->n % 4 == 0 && h->m % 4 == 0;
    if (h->transposed && !h->tc_ok) L.dbarT = take(cnt * m * n * 4);   // the node mean in storage orientation, before it is transposed
    if (h->tc_ok) {
        const size_t ncp = align_up(ell, 16);
        L.dbarT = take(cnt * m * n * 4);
        L.Yt = take(cnt * ell * m * 4);
        L.Zt = take(cnt * ell * n * 4);
        size_t g1 = gemm_tc_splits(h->m, h->n, h->count, h->sm_count) * cnt * m * ncp;
        size_t g2 = gemm_tc_splits(h->n, h->m, h->count, h->sm_count) * cnt * n * ncp;
        h->gpart_floats = std::max(g1, g2);
        L.gpart = take(h->gpart_floats * 4);
    }
    // ---- projection on the tensor cores (r > 16, or refresh blocks of 17..128 columns) ----
    h->ptc_ok = (h->r > 16 || ell > 16) && h->n % 4 == 0;
    // ... and the projection of the two-pass deferred mode (pending residual folded in as a tensor-core product), up to 32 columns
    h->ppt_ok = h->mode == 1 && h->r <= 32 && h->n % 4 == 0 && !h->transposed && !h->grad_bf16 && h->power_steps == 1 && h->pend_tc != 2;
    h->ptc_ncp = h->ptc_ok ? (int)align_up(std::min<size_t>(128, std::max(r, ell)), 16) : 0;
    if (h->ptc_ok || h->ppt_ok) {
        const size_t ncp = std::max<size_t>(h->ptc_ncp, h->ppt_ok ? align_up(r, 16) : 0);
        L.ptQ = take(3 * cnt * ncp * align_up(std::max(m, n), TC_BK) * 4);   // split Q^T (projection) or P~^T (back-projection)
    }
    if (h->ppt_ok) {
        L.ppP = take(cnt * align_up(m, TC_BM) * 2 * TC_BK * 4);         // two terms of P~_prev, one image per 128-row block
        L.ppQ = take(cnt * N * align_up(n, TC_BK) * 3 * TC_BK * 4);     // three terms of Qsub, one image per 32-column block
    }
    // ---- residual update on the tensor cores: split (head + tail) padded copies of P~ and Q_i ----
    h->rtc_ok = h->r > 16 && h->n % 4 == 0;
    if (h->rtc_ok) {
        h->rtc_KP = (int)align_up(r, TC_BK);
        const size_t KP = h->rtc_KP;
        L.rtP = take(3 * cnt * m * KP * 4);       // the three TF32 terms of P~, padded to KP columns
        L.rtQ = take(3 * cnt * N * n * KP * 4);   // the same for Q_i
    }
    // ---- single-pass mode ----
    // A CTA owns WC in {128, 256, 512} columns of every node; the tile of S it keeps on chip and the
    // registers of its back-projection bound N * WC by 2048.  CS = ceil(n / WC) CTAs form a cluster.
    h->fused_ok = false;
    if (h->mode == 1 && h->r <= 8 && h->n % 4 == 0 && h->N <= 16 && !h->transposed) {
        const int RP = h->r <= 4 ? 4 : 8;
        const int wcmax = h->N <= 4 ? 512 : (h->N <= 8 ? 256 : 128);
        int bestWC = 0, bestCS = 0;
        int64_t bestWaste = -1;
        for (int WC = 128; WC <= wcmax; WC *= 2) {
            int CS = ceil_div(h->n, WC);
            if (CS > FU_MAXCS) continue;
            int64_t waste = (int64_t)CS * WC - h->n;
            if (bestWaste < 0 || waste <= bestWaste) { bestWaste = waste; bestWC = WC; bestCS = CS; }
        }
        if (bestWC) {
            h->fused_ok = true; h->RP = RP; h->CS = bestCS; h->WC = bestWC;
            h->fused_smem = RP == 4 ? (bestWC == 128 ? fused_smem_bytes<4, 128>(h->N) : bestWC == 256 ? fused_smem_bytes<4, 256>(h->N) : fused_smem_bytes<4, 512>(h->N))
                                    : (bestWC == 128 ? fused_smem_bytes<8, 128>(h->N) : bestWC == 256 ? fused_smem_bytes<8, 256>(h->N) : fused_smem_bytes<8, 512>(h->N));
            h->nblk = ceil_div(h->m, FU_R);
            // Row slots per matrix.  The workspace is sized here, on the host, for KCmax slots from a table of
            // the clusters of each size that a B200 keeps resident (one CTA per SM); the first launch asks the
            // device for the real number and picks KC <= KCmax for whole waves.
            // (upper bound for sizing: one CTA per multiprocessor, clusters packed without regard to the GPC borders)
            const int resident = std::max(1, h->sm_count / bestCS);
            h->KCmax = (int)std::max<int64_t>(1, std::min<int64_t>(std::min(std::max(1, h->nblk / 4), 64),
                                                                   (16 * resident + h->count - 1) / h->count));
            h->KC = h->KCmax;
            h->active_clusters = -1;
        }
    }
    // ---- L2-pipelined single-pass kernel: up to 16 columns, 16-byte row strides ----
    // Which kernel serves the SSP steps of the deferred mode (PSGD_OPT_SINGLE_PASS).  Measured on a B200: up to 4 columns the
    // cluster kernel is the fastest everywhere (0.76 of the 12 B/element roofline on 16384 x 4096, N = 4).  From 5 to 8
    // columns it still is where its clusters are small enough to fill the chip (3 CTAs for n = 768: 2.06 against 2.21 ms per
    // step of the 130M-shaped stack), while with clusters of more than 4 CTAs (8 for n = 4096: 120 of 148 multiprocessors
    // busy) the two-pass kernels win (0.86 against 1.04 ms).  Above 8 columns the two-pass kernels are the fastest.
    if (h->single_pass_kernel == 2 || (h->single_pass_kernel == 0 && h->r > 4 && h->CS > 4 && !h->grad_bf16)) h->fused_ok = false;
    h->stream_ok = !h->transposed && h->mode == 1 && h->single_pass_kernel == 3 && h->r <= 16 && h->n % 4 == 0 && h->N <= 16 && !h->grad_bf16;
    size_t wslots = h->fused_ok ? (size_t)h->KCmax : 0;
    if (h->stream_ok) {
        if (!h->fused_ok) h->RP = h->r <= 4 ? 4 : (h->r <= 8 ? 8 : 16);
        h->s_nrb = ceil_div(h->m, SS_ROWS);
        h->s_ngrp = ceil_div(h->s_nrb, SS_GROUP);
        const int ntiles = ceil_div(h->n, SS_TCOLS);
        h->s_tpu = std::min(SS_MAXTPU, ntiles);
        h->s_csplit = ceil_div(ntiles, h->s_tpu);
        h->s_CB = ceil_div(h->n, SS_BCOLS);
        // row slots per (matrix, node, column block): as many as there are back-projection workers to take them
        const int64_t pairs = (int64_t)h->count * h->N * h->s_CB;
        const int64_t workers = (int64_t)(4 - (h->RP >= 16 ? 2 : 3)) * h->sm_count;     // 4 - stream_groups<RP>() per CTA
        h->s_KC = (int)std::max<int64_t>(1, std::min<int64_t>(std::min(h->s_ngrp, 32), workers / pairs));
        h->s_grid = -1;
        wslots = std::max<size_t>(wslots, 2 * (size_t)h->s_KC);
    }
    if (h->fused_ok || h->stream_ok) {
        const size_t RP = h->RP, KC = wslots;
        L.Qpad = take(cnt * n * RP * 4);
        L.Ppad = take(cnt * m * RP * 4);
        L.Qsub = take(cnt * N * n * RP * 4);
        L.Tacc = take(cnt * RP * RP * 4);
        L.Pout = take(cnt * m * RP * 4);
        L.Wpart = take(cnt * KC * N * n * RP * 4);
        L.Cmat = take(cnt * RP * RP * 4);
        L.Cpart = take(cnt * (size_t)ceil_div(h->n, 16) * RP * RP * 8);
    }
    if (h->stream_ok) {
        L.sPpart = take(cnt * (size_t)h->s_nrb * N * h->s_csplit * SS_ROWS * h->RP * 4);
        L.sCnt = take(cnt * (size_t)h->s_nrb * 2 * 4);
        L.sGram = take(cnt * (size_t)h->s_nrb * r * r * 8);
    }
    L.total = off;
}

#define PSGD_CUDA(h, call)                                                                  \
    do {                                                                                    \
        cudaError_t e_ = (call);                                                            \
        if (e_ != cudaSuccess) {                                                            \
            snprintf((h)->err, sizeof((h)->err), "%s: %s", #call, cudaGetErrorString(e_));  \
            return PSGD_E_CUDA;                                                             \
        }                                                                                   \
    } while (0)

struct Launcher {
    psgd_handle* h;
    cudaStream_t st;
    psgd_status status = PSGD_OK;
    int force_kind = -1;  // when >= 0 every launch is booked under this family
    void begin(int kind) {
        if (!h->profiling) return;
        ProfEvent ev;
        ev.kind = force_kind >= 0 ? force_kind : kind;
        cudaEventCreate(&ev.a);
        cudaEventCreate(&ev.b);
        cudaEventRecord(ev.a, st);
        h->events.push_back(ev);
    }
    void check(cudaError_t e) {   // a runtime call that is not a launch of this library's kernels
        if (e != cudaSuccess && status == PSGD_OK) {
            snprintf(h->err, sizeof(h->err), "runtime call: %s", cudaGetErrorString(e));
            status = PSGD_E_CUDA;
        }
    }
    void end() {
        if (h->profiling) cudaEventRecord(h->events.back().b, st);
        h->launches++;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess && status == PSGD_OK) {
            snprintf(h->err, sizeof(h->err), "kernel launch: %s", cudaGetErrorString(e));
            status = PSGD_E_CUDA;
        }
    }
};

// Opt a kernel in to `bytes` of dynamic shared memory: the attribute is set once per (device, kernel) and raised
// only when a larger size is asked for.
void set_smem_attr(const void* kernel, size_t bytes) {
    static std::mutex mu;
    static std::map<std::pair<int, const void*>, size_t> done;
    int dev = 0;
    cudaGetDevice(&dev);
    std::lock_guard<std::mutex> lock(mu);
    size_t& have = done[std::make_pair(dev, kernel)];
    if (bytes > have) {
        cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
        have = bytes;
    }
}
template <typename K>
void allow_smem(K kernel, size_t bytes) {
    if (bytes > 48 * 1024) set_smem_attr((const void*)kernel, bytes);
}

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// ---- TMA tensor maps ----------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}
// Rank-3 map over [count*N][m][n] float32 with tiles of `rows` rows x bw columns of one node; out-of-range reads give zeros.
bool encode_tile_map(CUtensorMap* map, const void* base, int64_t n, int64_t m, int64_t mats, int bw, int rows,
                     CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE, bool bf16 = false) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t es = bf16 ? 2 : 4;
    cuuint64_t dims[3] = {(cuuint64_t)n, (cuuint64_t)m, (cuuint64_t)mats};
    cuuint64_t strides[2] = {(cuuint64_t)n * es, (cuuint64_t)m * (cuuint64_t)n * es};
    cuuint32_t box[3] = {(cuuint32_t)bw, (cuuint32_t)rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same through the handle's cache: a descriptor is encoded once per distinct (pointer, shape, tile) and reused by
// every later launch (E, Q and the workspace keep their addresses; gradient buffers usually alternate between a few).
bool make_tile_map(psgd_handle* h, CUtensorMap* map, const void* base, int64_t n, int64_t m, int64_t mats, int bw, int rows,
                   CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_NONE, bool bf16 = false) {
    for (const CachedMap& c : h->maps)
        if (c.base == base && c.n == n && c.m == m && c.mats == mats && c.bw == bw && c.rows == rows && c.swizzle == (int)swizzle &&
            c.bf16 == (bf16 ? 1 : 0)) {
            *map = c.map;
            return true;
        }
    CachedMap c{base, n, m, mats, bw, rows, (int)swizzle, bf16 ? 1 : 0, {}};
    if (!encode_tile_map(&c.map, base, n, m, mats, bw, rows, swizzle, bf16)) return false;
    *map = c.map;
    constexpr size_t kMaxCached = 96;
    if (h->maps.size() < kMaxCached) h->maps.push_back(c);
    else { h->maps[h->map_next] = c; h->map_next = (h->map_next + 1) % kMaxCached; }
    return true;
}


// C = A B^T on the tensor cores: A [count][M][K], B [count][Nc][K] (both K-major), C [count][M][Nc].
void launch_gemm_tc(Launcher& L, psgd_handle* h, const float* A, const float* B, float* C, int M, int Nc, int K, int kind) {
    const int cnt = h->count;
    const int Ncp = (int)align_up(Nc, 16);
    const int KB = ceil_div(K, TC_BK);
    const int S = gemm_tc_splits(M, K, cnt, h->sm_count);
    const int kbps = ceil_div(KB, S);
    float* Cpart = (float*)(h->ws + h->lay.gpart);
    if ((size_t)cnt * S * M * Ncp > h->gpart_floats) { L.status = PSGD_E_WORKSPACE; return; }
    CUtensorMap tmA, tmB;
    if (!make_tile_map(h, &tmA, A, K, M, cnt, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tile_map(h, &tmB, B, K, Nc, cnt, TC_BK, Ncp, CU_TENSOR_MAP_SWIZZLE_128B)) {
        snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
        L.status = PSGD_E_CUDA;
        return;
    }
    GemmTcArgs g{Cpart, M, Ncp, K, S, kbps, (int*)(h->ws + h->lay.flags)};
    size_t smem = gemm_tc_smem_bytes(Ncp);
    set_smem_attr((const void*)k_gemm_tf32, smem);
    L.begin(kind);
    k_gemm_tf32<<<dim3(ceil_div(M, TC_BM), S, cnt), TC_THREADS, smem, L.st>>>(tmA, tmB, g);
    L.end();
    size_t tot = (size_t)cnt * M * Nc;
    L.begin(kind);
    k_gemm_reduce<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Cpart, C, M, Nc, Ncp, S, cnt);
    L.end();
}

// M = G + E over E (Eq. (7a)), optionally Dbar = node mean of M (SVD-Comp, first line): 128-bit accesses when the
// row-major arrays allow it.
void launch_add_mean(Launcher& L, const void* G, bool bf16, float* E, float* dbar, size_t per_mat, int N, int cnt, int kind) {
    const bool vec = per_mat % 4 == 0 && aligned16(E) && (!dbar || aligned16(dbar)) && (((uintptr_t)G & (bf16 ? 7 : 15)) == 0);
    const int V = vec ? 4 : 1;
    const size_t want = (per_mat + (size_t)V * 256 - 1) / ((size_t)V * 256);
    const unsigned gx = (unsigned)std::max<size_t>(1, std::min<size_t>(want, (size_t)std::max(1, L.h->sm_count * 8 / cnt)));
    dim3 grid(gx, (unsigned)cnt);
    L.begin(kind);
    if (bf16) {
        if (vec) k_add_mean<unsigned short, 4><<<grid, 256, 0, L.st>>>((const unsigned short*)G, E, dbar, per_mat, N, cnt);
        else k_add_mean<unsigned short, 1><<<grid, 256, 0, L.st>>>((const unsigned short*)G, E, dbar, per_mat, N, cnt);
    } else {
        if (vec) k_add_mean<float, 4><<<grid, 256, 0, L.st>>>((const float*)G, E, dbar, per_mat, N, cnt);
        else k_add_mean<float, 1><<<grid, 256, 0, L.st>>>((const float*)G, E, dbar, per_mat, N, cnt);
    }
    L.end();
}

// ---- K1 dispatch ------------------------------------------------------------
template <int RP, int VEC, bool ADD, bool STORE>
void launch_project_t(Launcher& L, const ProjectArgs& a, int count) {
    auto kern = k_project<RP, VEC, ADD, STORE>;
    size_t smem = project_smem_bytes<RP, ADD>();
    allow_smem(kern, smem);
    dim3 grid(ceil_div(a.rows, PJ_TR), a.nodes, count * a.nchunks);
    L.begin(PSGD_K_PROJECT);
    kern<<<grid, PJ_THREADS, smem, L.st>>>(a);
    L.end();
}
template <int RP>
void launch_project_rp(Launcher& L, const ProjectArgs& a, int count, bool vec, bool add) {
    if (vec) {
        if (add) launch_project_t<RP, 4, true, true>(L, a, count);
        else launch_project_t<RP, 4, false, false>(L, a, count);
    } else {
        if (add) launch_project_t<RP, 1, true, true>(L, a, count);
        else launch_project_t<RP, 1, false, false>(L, a, count);
    }
}
// P = (G + (Delta_prev - P~_prev Qsub^T)) Q, M = G + e stored over Delta_prev: the projection of the two-pass deferred
// mode (r <= 16, one chunk of columns).
void launch_project_pending(Launcher& L, const float* G, float* E, const float* Q, float* P, const float* Pprev, const float* Qsub,
                            int qsub_per_node, int rows, int n, int r, int nodes, int count, bool vec) {
    ProjectArgs a{G, E, E, Q, P, rows, n, r, nodes, 1, nullptr};
    a.Pprev = Pprev; a.Qsub = Qsub; a.qsub_per_node = qsub_per_node;
    vec = vec && aligned16(G) && aligned16(E);
    dim3 grid(ceil_div(rows, PJ_TR), nodes, count);
    auto go = [&](auto kern, size_t smem) {
        allow_smem(kern, smem);
        L.begin(PSGD_K_PROJECT);
        kern<<<grid, PJ_THREADS, smem, L.st>>>(a);
        L.end();
    };
    if (r <= 4) { if (vec) go(k_project<4, 4, true, true, true>, project_smem_bytes<4, true, true>()); else go(k_project<4, 1, true, true, true>, project_smem_bytes<4, true, true>()); }
    else if (r <= 8) { if (vec) go(k_project<8, 4, true, true, true>, project_smem_bytes<8, true, true>()); else go(k_project<8, 1, true, true, true>, project_smem_bytes<8, true, true>()); }
    else { if (vec) go(k_project<16, 4, true, true, true>, project_smem_bytes<16, true, true>()); else go(k_project<16, 1, true, true, true>, project_smem_bytes<16, true, true>()); }
}

// K splits of the tensor-core projection: one CTA per multiprocessor runs at a time, so a grid that ends in a short last
// wave leaves most of the chip idle for a whole row block; two CTAs per row block (half of the columns each) make the waves
// twice as many and half as long.  Cost model: waves x (K blocks per CTA + a fixed cost for filling and draining its rings).
int proj_tc_ksplit(int tiles, int KB, int sms) {
    if (KB < 16) return 1;
    const long long c1 = (long long)ceil_div(tiles, sms) * (KB + 8), c2 = (long long)ceil_div(2 * tiles, sms) * (KB / 2 + 8);
    return c2 * 100 < c1 * 97 ? 2 : 1;
}

// Tensor-core form for more than 16 columns (exactly split TF32 products, see psgd_gemm_tc.cuh).
bool launch_project_tc(Launcher& L, const float* A, const float* B, float* Mout, const float* Q, float* P, int rows, int n,
                       int r, int nodes, int count, const int* skip) {
    psgd_handle* h = L.h;
    const int Ncp = (int)align_up(r, 16);
    // (n is the row length of the matrices handed in, which with transposed storage is not the handle's n: 16-byte rows for TMA)
    if (!h->ptc_ok || Ncp > h->ptc_ncp || r > 128 || n % 4 != 0 || !aligned16(A) || (B && !aligned16(B)) || (Mout && !aligned16(Mout))) return false;
    const int mats = count * nodes;
    float* Qimg = (float*)(h->ws + h->lay.ptQ);
    const int KB = ceil_div(n, TC_BK);
    const size_t tot = (size_t)count * KB * Ncp * TC_BK;
    L.begin(PSGD_K_PROJECT);
    k_split_img_t<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Q, Qimg, n, r, Ncp, KB, count, skip);
    L.end();
    CUtensorMap tA, tB;
    bool ok = make_tile_map(h, &tA, A, n, rows, mats, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B) &&
              make_tile_map(h, &tB, B ? B : A, n, rows, mats, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (!ok) {
        snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
        L.status = PSGD_E_CUDA;
        return true;
    }
    ProjTcArgs a{B ? Mout : nullptr, P, rows, n, r, Ncp, proj_tc_nh(Ncp), B ? 1 : 0, nodes, (int*)(h->ws + h->lay.flags), skip};
    size_t smem = proj_tc_smem_bytes(Ncp);
    set_smem_attr((const void*)k_project_tc<false>, smem);
    // (a launch that a device-side flag may skip must leave P alone: no zeroing, hence no split)
    const int KS = skip ? 1 : proj_tc_ksplit(ceil_div(rows, TC_BM) * mats, KB, h->sm_count);
    if (KS > 1) L.check(cudaMemsetAsync(P, 0, (size_t)mats * rows * r * 4, L.st));
    L.begin(PSGD_K_PROJECT);
    k_project_tc<false><<<dim3(ceil_div(rows, TC_BM), mats, KS), PT_THREADS, smem, L.st>>>(tA, tB, Qimg, a);
    L.end();
    return true;
}

// The projection of the two-pass deferred mode on the tensor cores (up to 32 columns): P = (G + (Delta_prev - P~_prev Qsub^T)) Q,
// M stored over Delta_prev.  False when the shape or the pointers do not allow it (nothing has been launched then).
bool launch_project_pending_tc(Launcher& L, const float* G, float* E, const float* Q, float* P, const float* Pprev, const float* Qsub,
                               int qsub_per_node, int rows, int n, int r, int nodes, int count) {
    psgd_handle* h = L.h;
    if (!h->ppt_ok || r > 32 || !aligned16(G) || !aligned16(E)) return false;
    const int Ncp = (int)align_up(r, 16);
    const int mats = count * nodes, qmats = qsub_per_node ? mats : count;
    const int KB = ceil_div(n, TC_BK), RT = ceil_div(rows, TC_BM);
    float* Qimg = (float*)(h->ws + h->lay.ptQ);
    float* Pimg = (float*)(h->ws + h->lay.ppP);
    float* QSimg = (float*)(h->ws + h->lay.ppQ);
    CUtensorMap tA, tB;
    if (!make_tile_map(h, &tA, G, n, rows, mats, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tile_map(h, &tB, E, n, rows, mats, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B)) {
        snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
        L.status = PSGD_E_CUDA;
        return true;
    }
    const int GQ = r <= 8 ? 4 : (r <= 16 ? 2 : 1), groups = ceil_div(KB, GQ);     // K blocks whose rank columns share one image of Qsub
    const size_t tq = (size_t)count * KB * Ncp * TC_BK, tp = (size_t)count * RT * TC_BM * TC_BK, ts = (size_t)qmats * groups * 32 * TC_BK;
    L.begin(PSGD_K_PROJECT);
    k_split_img_t<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(Q, Qimg, n, r, Ncp, KB, count, nullptr);
    L.end();
    L.begin(PSGD_K_PROJECT);
    k_split_img_rows<<<(unsigned)((tp + 255) / 256), 256, 0, L.st>>>(Pprev, Pimg, rows, r, TC_BM, 2, count);
    L.end();
    L.begin(PSGD_K_PROJECT);
    k_split_img_qs<<<(unsigned)((ts + 255) / 256), 256, 0, L.st>>>(Qsub, QSimg, n, r, GQ, groups, qmats);
    L.end();
    ProjTcArgs a{E, P, rows, n, r, Ncp, proj_tc_nh(Ncp, true), 1, nodes, (int*)(h->ws + h->lay.flags), nullptr,
                 Pimg, QSimg, qsub_per_node, ceil_div(r, 8), GQ, groups};
    size_t smem = proj_tc_smem_bytes(Ncp, true);
    set_smem_attr((const void*)k_project_tc<true>, smem);
    const int KS = proj_tc_ksplit(RT * mats, KB, h->sm_count);
    if (KS > 1) L.check(cudaMemsetAsync(P, 0, (size_t)mats * rows * r * 4, L.st));
    L.begin(PSGD_K_PROJECT);
    k_project_tc<true><<<dim3(RT, mats, KS), PT_THREADS_PEND, smem, L.st>>>(tA, tB, Qimg, a);
    L.end();
    return true;
}

// P = (A [+B]) Q for all matrices; `add` also stores A+B into Mout.
void launch_project(Launcher& L, const float* A, const float* B, float* Mout, const float* Q, float* P, int rows, int n,
                    int r, int nodes, int count, bool vec, const int* skip = nullptr) {
    if (r > 16 && launch_project_tc(L, A, B, Mout, Q, P, rows, n, r, nodes, count, skip)) return;
    ProjectArgs a{A, B, Mout, Q, P, rows, n, r, nodes, 1, skip};
    bool add = B != nullptr;
    vec = vec && aligned16(A) && (!B || aligned16(B)) && (!Mout || aligned16(Mout));
    if (r <= 4) launch_project_rp<4>(L, a, count, vec, add);
    else if (r <= 8) launch_project_rp<8>(L, a, count, vec, add);
    else if (r <= 16) launch_project_rp<16>(L, a, count, vec, add);
    else {
        a.nchunks = ceil_div(r, 32);
        // the in-place store of A+B is only safe when a single CTA reads each tile
        launch_project_rp<32>(L, a, count, vec, add && a.nchunks == 1);
    }
}

// ---- K3 dispatch ------------------------------------------------------------
template <int RP>
void launch_back_rp(Launcher& L, BackArgs a, int mats, bool vec) {
    a.nchunks = ceil_div(a.r, RP);
    dim3 grid(ceil_div(a.n, BP_COLS), a.S, mats * a.nchunks);
    L.begin(PSGD_K_BACKPROJECT);
    if (vec) k_backproject<RP, 4><<<grid, BP_THREADS, 0, L.st>>>(a);
    else k_backproject<RP, 1><<<grid, BP_THREADS, 0, L.st>>>(a);
    L.end();
}
// Tensor-core form for more than 16 columns (M as the MN-major operand, see psgd_gemm_tc.cuh).  Picks its own number of
// row splits (at most S, the number the partial buffer was sized for) and returns it, 0 if the shape is not eligible.
int launch_back_tc(Launcher& L, const float* M, const float* Phat, float* part, int rows, int n, int r, int nodes, int count,
                   int S, const int* skip) {
    psgd_handle* h = L.h;
    const int Ncp = (int)align_up(r, 16);
    if (!h->ptc_ok || Ncp > h->ptc_ncp || r > 128 || n % 4 != 0 || !aligned16(M)) return 0;
    const int mats = count * nodes;
    const int KB = ceil_div(rows, TC_BK);
    const int64_t base = (int64_t)ceil_div(n, TC_BM) * mats;
    int best = 1;
    int64_t best_cost = -1;
    for (int s = 1; s <= std::min(S, 32); ++s) {       // cost: waves x (K blocks per CTA + fixed start-up and epilogue)
        const int kbs = ceil_div(KB, s);
        if (s > 1 && kbs < 16) break;
        if ((int64_t)(s - 1) * kbs >= KB) continue;     // would leave an empty split
        const int64_t cost = ((base * s + h->sm_count - 1) / h->sm_count) * (kbs + 10);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    const int St = best, kbs = ceil_div(KB, St);
    float* Pimg = (float*)(h->ws + h->lay.ptQ);        // P~^T as one shared-memory image per K block of 32 rows
    const size_t tot = (size_t)count * KB * Ncp * TC_BK;
    L.begin(PSGD_K_BACKPROJECT);
    k_split_img_t<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Phat, Pimg, rows, r, Ncp, KB, count, skip);
    L.end();
    CUtensorMap tM;
    bool ok = make_tile_map(h, &tM, M, n, rows, mats, 32, TC_BK, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B);
    if (!ok) {
        snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
        L.status = PSGD_E_CUDA;
        return St;
    }
    BackTcArgs a{part, rows, n, r, Ncp, back_tc_nh(Ncp), St, kbs, nodes, (int*)(h->ws + h->lay.flags), skip};
    size_t smem = back_tc_smem_bytes(Ncp);
    set_smem_attr((const void*)k_backproject_tc, smem);
    L.begin(PSGD_K_BACKPROJECT);
    k_backproject_tc<<<dim3(ceil_div(n, TC_BM), St, mats), PT_THREADS, smem, L.st>>>(tM, Pimg, a);
    L.end();
    return St;
}

// Q_i partial sums for all matrices; returns the number of row splits written (the S to hand to k_reduce_q).
int launch_back(Launcher& L, const float* M, const float* Phat, float* part, int rows, int n, int r, int nodes,
                 int count, int rpc, int S, bool vec, const int* gate = nullptr, const int* skip = nullptr) {
    if (r > 16 && !gate) {
        const int St = launch_back_tc(L, M, Phat, part, rows, n, r, nodes, count, S, skip);
        if (St > 0) return St;
    }
    BackArgs a{M, Phat, part, rows, n, r, nodes, 1, rpc, S, gate, skip};
    vec = vec && aligned16(M);
    // 4, 8 or 16 columns exactly, whole 256-column blocks of 16-byte aligned rows: tiles of M staged by TMA
    if (!gate && vec && (r == 4 || r == 8 || r == 16) && n >= BP_COLS && rpc % BQ_ROWS == 0 && aligned16(Phat) && L.h->bq_ok) {
        CUtensorMap tM;
        if (make_tile_map(L.h, &tM, M, n, rows, (int64_t)count * nodes, BP_COLS, BQ_ROWS)) {
            // row chunks: two CTAs per multiprocessor run at a time; fewest waves x (tiles per CTA + start-up), at most the S
            // chunks the partial buffer was sized for
            const int64_t base = (int64_t)ceil_div(n, BP_COLS) * count * nodes, slots = 2 * (int64_t)L.h->sm_count;
            int bestS = S, best_rpc = rpc;
            int64_t best_cost = -1;
            for (int s2 = 1; s2 <= S; ++s2) {
                const int rpc2 = (int)align_up(ceil_div(rows, s2), BP_SUB), sc = ceil_div(rows, rpc2);
                const int64_t cost = ((base * sc + slots - 1) / slots) * (ceil_div(rpc2, BQ_ROWS) + 3);
                if (best_cost < 0 || cost < best_cost) { best_cost = cost; bestS = sc; best_rpc = rpc2; }
            }
            S = bestS;
            a.S = S; a.rows_per_chunk = best_rpc;
            dim3 grid(ceil_div(n, BP_COLS), S, count * nodes);
            int* flags = (int*)(L.h->ws + L.h->lay.flags);
            auto go = [&](auto kern, size_t smem) {
                set_smem_attr((const void*)kern, smem);
                L.begin(PSGD_K_BACKPROJECT);
                kern<<<grid, BQ_THREADS, smem, L.st>>>(tM, a, flags);
                L.end();
            };
            if (r == 4) go(k_backproject_tma<4>, backq_smem_bytes<4>());
            else if (r == 8) go(k_backproject_tma<8>, backq_smem_bytes<8>());
            else go(k_backproject_tma<16>, backq_smem_bytes<16>());
            return S;
        }
    }
    if (r <= 4) launch_back_rp<4>(L, a, count * nodes, vec);
    else if (r <= 8) launch_back_rp<8>(L, a, count * nodes, vec);
    else launch_back_rp<16>(L, a, count * nodes, vec);
    return S;
}

// ---- K4 dispatch ------------------------------------------------------------
// Tensor-core form for ranks above 16 (exactly split TF32 rank-r product in tensor memory, see psgd_gemm_tc.cuh).
bool launch_resid_tc(Launcher& L, const float* M, float* Out, const float* Phat, const float* Qf, int rows, int n, int r,
                     int nodes, int mats, int q_per_node, int out_per_node) {
    psgd_handle* h = L.h;
    if (!h->rtc_ok || n % 4 != 0 || !aligned16(Out) || (M && !aligned16(M))) return false;
    const int KP = h->rtc_KP, cnt = h->count;
    const int qmats = q_per_node ? mats : cnt;
    // the split copies of the factors were sized for the handle's own orientation (rows = m, Q_i per node of n rows)
    if (rows > h->m || (int64_t)qmats * n > (int64_t)cnt * h->N * h->n) return false;
    const size_t tp = (size_t)cnt * rows * KP, tq = (size_t)qmats * n * KP;
    float* Pt[3] = {(float*)(h->ws + h->lay.rtP), (float*)(h->ws + h->lay.rtP) + tp, (float*)(h->ws + h->lay.rtP) + 2 * tp};
    float* Qt[3] = {(float*)(h->ws + h->lay.rtQ), (float*)(h->ws + h->lay.rtQ) + tq, (float*)(h->ws + h->lay.rtQ) + 2 * tq};
    L.begin(PSGD_K_RESIDUAL);
    k_split_pad<<<(unsigned)((tp + 255) / 256), 256, 0, L.st>>>(Phat, Pt[0], Pt[1], Pt[2], (size_t)cnt * rows, r, KP);
    L.end();
    L.begin(PSGD_K_RESIDUAL);
    k_split_pad<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(Qf, Qt[0], Qt[1], Qt[2], (size_t)qmats * n, r, KP);
    L.end();
    CUtensorMap tP[3], tQ[3];
    for (int t = 0; t < 3; ++t) {
        if (!make_tile_map(h, &tP[t], Pt[t], KP, rows, cnt, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
            !make_tile_map(h, &tQ[t], Qt[t], KP, n, qmats, TC_BK, RT_BN, CU_TENSOR_MAP_SWIZZLE_128B)) {
            snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
            L.status = PSGD_E_CUDA;
            return true;
        }
    }
    ResidTcArgs a{M, Out, rows, n, KP, out_per_node ? nodes : 1, q_per_node, (int*)(h->ws + h->lay.flags)};
    size_t smem = resid_tc_smem_bytes();
    set_smem_attr((const void*)k_residual_tc, smem);
    L.begin(PSGD_K_RESIDUAL);
    k_residual_tc<<<dim3(ceil_div(rows, TC_BM), mats), RT_THREADS, smem, L.st>>>(tP[0], tP[1], tP[2], tQ[0], tQ[1], tQ[2], a);
    L.end();
    return true;
}

void launch_resid(Launcher& L, const float* M, float* Out, const float* Phat, const float* Qf, int rows, int n, int r,
                  int nodes, int mats, int q_per_node, int out_per_node, bool vec, int p_per_node = 0) {
    if (r > 16 && !p_per_node && launch_resid_tc(L, M, Out, Phat, Qf, rows, n, r, nodes, mats, q_per_node, out_per_node)) return;
    int rpc = 128;
    while (rpc > RS_SUB && (int64_t)mats * ceil_div(n, RS_COLS) * ceil_div(rows, rpc) < 4 * L.h->sm_count) rpc /= 2;
    ResidArgs a{M, Out, Phat, Qf, rows, n, r, nodes, rpc, q_per_node, out_per_node};
    a.p_per_node = p_per_node;
    vec = vec && aligned16(Out) && (!M || aligned16(M));
    dim3 grid(ceil_div(n, RS_COLS), ceil_div(rows, rpc), mats);
    L.begin(PSGD_K_RESIDUAL);
    if (r <= 4) { if (vec) k_residual<4, 4><<<grid, RS_THREADS, 0, L.st>>>(a); else k_residual<4, 1><<<grid, RS_THREADS, 0, L.st>>>(a); }
    else if (r <= 8) { if (vec) k_residual<8, 4><<<grid, RS_THREADS, 0, L.st>>>(a); else k_residual<8, 1><<<grid, RS_THREADS, 0, L.st>>>(a); }
    else { if (vec) k_residual<16, 4><<<grid, RS_THREADS, 0, L.st>>>(a); else k_residual<16, 1><<<grid, RS_THREADS, 0, L.st>>>(a); }
    L.end();
}

// Momentum-SGD hand-off (Eq. (7c)): mom <- mu mom + P~ Q^T, X <- X - eta mom, the reconstruction never stored.
void launch_msgd(Launcher& L, float* X, float* Mom, float eta, float mu, const float* Phat, const float* Qf, int rows, int n,
                 int r, int mats) {
    int rpc = 128;
    while (rpc > RS_SUB && (int64_t)mats * ceil_div(n, RS_COLS) * ceil_div(rows, rpc) < 4 * L.h->sm_count) rpc /= 2;
    ResidArgs a{nullptr, nullptr, Phat, Qf, rows, n, r, 1, rpc, 0, 0};
    a.X = X; a.Mom = Mom; a.eta = eta; a.mu = mu;
    dim3 grid(ceil_div(n, RS_COLS), ceil_div(rows, rpc), mats);
    L.begin(PSGD_K_RESIDUAL);
    if (r <= 4) k_residual<4, 1><<<grid, RS_THREADS, 0, L.st>>>(a);
    else if (r <= 8) k_residual<8, 1><<<grid, RS_THREADS, 0, L.st>>>(a);
    else k_residual<16, 1><<<grid, RS_THREADS, 0, L.st>>>(a);
    L.end();
}

// ---- K2: X <- orthonormal factor of X (rows x c), in place or into Xout ------
void launch_orth(Launcher& L, psgd_handle* h, const float* X, float* Xout, int rows, int c, int kind, float* XoutT = nullptr,
                 bool complete = false, const int* skip = nullptr) {
    char* ws = h->ws;
    double* gram = (double*)(ws + h->lay.gram);
    double* T = (double*)(ws + h->lay.T);
    int* flags = (int*)(ws + h->lay.flags);
    int nparts = ceil_div(rows, GR_ROWS);
    int nblk = ceil_div(c, 64);
    GramArgs g{X, gram, rows, c, nparts, nullptr, skip};
    L.begin(kind);
    k_gram<<<dim3(nparts, nblk * nblk, h->count), 256, 0, L.st>>>(g);
    L.end();
    if (nparts > 4) {   // fold the partials in parallel first; the Cholesky kernel then reads partial 0 with the original stride
        size_t tot = (size_t)c * c * h->count;
        L.begin(kind);
        k_gram_sum<<<(unsigned)((tot + 31) / 32), 256, 0, L.st>>>(gram, c * c, nparts, h->count, skip);
        L.end();
    }
    size_t smem = (size_t)c * chol_ld(c) * 8;
    L.begin(kind);
    int* defic = (int*)(ws + h->lay.defic);
    const int np = nparts > 4 ? -nparts : nparts;
    int* dfc = complete ? defic : nullptr;
    // wide CTAs only while every matrix has a multiprocessor to itself: with more matrices than that the narrow ones share
    // the multiprocessors and finish sooner together
    const int nt = h->count <= h->sm_count ? chol_threads(c) : 256;
    if (nt == 1024) {
        allow_smem(k_chol_t<1024>, smem);
        k_chol_t<1024><<<h->count, 1024, smem, L.st>>>(gram, T, c, np, flags, nullptr, 0.0, dfc, skip);
    } else if (nt == 512) {
        allow_smem(k_chol_t<512>, smem);
        k_chol_t<512><<<h->count, 512, smem, L.st>>>(gram, T, c, np, flags, nullptr, 0.0, dfc, skip);
    } else {
        allow_smem(k_chol_t<256>, smem);
        k_chol_t<256><<<h->count, 256, smem, L.st>>>(gram, T, c, np, flags, nullptr, 0.0, dfc, skip);
    }
    L.end();
    ApplyArgs ap{X, T, Xout, rows, c, c, c, 1, XoutT, skip};
    L.begin(kind);
    k_apply<<<dim3(ceil_div(rows, 32), h->count), 256, (size_t)32 * c * 4, L.st>>>(ap);
    L.end();
    if (complete) {   // rank-deficient P: replace the rejected columns by an orthonormal completion (no-op otherwise)
        L.begin(kind);
        k_complete<<<h->count, 256, 0, L.st>>>(Xout, nullptr, defic, flags, rows, c, 0, h->seed + (uint64_t)h->t);
        L.end();
    }
}

// ---- Algorithm 1, common tail: Q_i, Q, residual, optional dense reconstruction --
// defer: leave Delta_t in the E buffer (two-pass deferred mode); the next projection or psgd_materialize_error forms e_{t+1}
void tail(Launcher& L, psgd_handle* h, float* D_hat, bool defer = false) {
    char* ws = h->ws;
    float* Phat = (float*)(ws + h->lay.Phat);
    float* Qnode = (float*)(ws + h->lay.Qnode);
    float* part = (float*)(ws + h->lay.part);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    const int Sb = launch_back(L, h->E, Phat, part, m, n, r, N, cnt, h->rpc, h->S, h->vec4);
    size_t tot = (size_t)cnt * n * r;
    L.begin(PSGD_K_BACKPROJECT);
    k_reduce_q<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(part, Qnode, h->Q, n, r, N, Sb, cnt);
    L.end();
    if (defer) {
        h->pending = true;
        h->pending_fused = false;
    }
    else if (h->error_form == 0)
        launch_resid(L, h->E, h->E, Phat, Qnode, m, n, r, N, cnt * N, 1, 1, h->vec4);
    else
        launch_resid(L, h->E, h->E, Phat, h->Q, m, n, r, N, cnt * N, 0, 1, h->vec4);
    if (D_hat) launch_resid(L, nullptr, D_hat, Phat, h->Q, m, n, r, N, cnt, 0, 0, h->vec4);
}

// ---- SSP-Comp (Algorithm 1, first function) ------------------------------------
// Which projection carries the pending residual of the two-pass deferred mode.  The tensor-core form does not depend on the
// number of columns; the float32 form costs 2r multiply-adds per element and is the faster one only for few columns.
bool pending_on_tc(const psgd_handle* h) {
    if (!h->ppt_ok) return false;
    return h->pend_tc == 1 || h->r > PENDING_TC_MIN_R;
}
// SSP steps of the deferred mode in two passes (the residual stays pending in E): up to 16 columns, or up to 32 on the tensor cores
bool two_pass_ok(const psgd_handle* h) {
    return h->mode == 1 && h->power_steps == 1 && !h->grad_bf16 && (h->r <= 16 || pending_on_tc(h));
}

void materialize(Launcher& L, psgd_handle* h);

// P_i = (G_i + e_i) Q_{t-1} for every node, M_i left in the E buffer
void ssp_project(Launcher& L, psgd_handle* h, const void* Gv) {
    char* ws = h->ws;
    float* Pnode = (float*)(ws + h->lay.Pnode);
    float* Phat = (float*)(ws + h->lay.Phat);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    const float* G = (const float*)Gv;
    if (h->pending) {        // two-pass deferred mode: E holds Delta_{t-1}; P~_{t-1} and Q_i of the last step are still in place
        float* Qnode = (float*)(ws + h->lay.Qnode);
        const float* Qsub = h->error_form == 0 ? Qnode : h->Q;
        const int per_node = h->error_form == 0 ? 1 : 0;
        h->ran_pending_tc = pending_on_tc(h) && launch_project_pending_tc(L, G, h->E, h->Q, Pnode, Phat, Qsub, per_node, m, n, r, N, cnt);
        if (!h->ran_pending_tc) {
            if (r > 16) {      // no float32 kernel folds a residual of more than 16 columns in: form it first (a third pass)
                materialize(L, h);
                ssp_project(L, h, Gv);
                return;
            }
            launch_project_pending(L, G, h->E, h->Q, Pnode, Phat, Qsub, per_node, m, n, r, N, cnt, h->vec4);
        }
    } else if (h->grad_bf16) {      // M = G + E formed in the E buffer first (10 B/element), then the projection reads M
        launch_add_mean(L, Gv, true, h->E, nullptr, (size_t)m * n, N, cnt, PSGD_K_PROJECT);
        launch_project(L, h->E, nullptr, nullptr, h->Q, Pnode, m, n, r, N, cnt, h->vec4);
    } else if (r <= 32 || (h->ptc_ok && aligned16(G))) {
        launch_project(L, G, h->E, h->E, h->Q, Pnode, m, n, r, N, cnt, h->vec4);
    } else {
        launch_add_mean(L, G, false, h->E, nullptr, (size_t)m * n, N, cnt, PSGD_K_PROJECT);
        launch_project(L, h->E, nullptr, nullptr, h->Q, Pnode, m, n, r, N, cnt, h->vec4);
    }
}

void ssp(Launcher& L, psgd_handle* h, const void* Gv) {
    char* ws = h->ws;
    float* Pnode = (float*)(ws + h->lay.Pnode);
    float* Pmean = (float*)(ws + h->lay.Pmean);
    float* Phat = (float*)(ws + h->lay.Phat);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    ssp_project(L, h, Gv);
    size_t tot = (size_t)cnt * m * r;
    L.begin(PSGD_K_ORTH);
    k_node_mean<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Pnode, Pmean, (size_t)m * r, N, cnt);
    L.end();
    launch_orth(L, h, Pmean, Phat, m, r, PSGD_K_ORTH, nullptr, true);
    // K-step power iteration (Eq. (8)): K - 1 more rounds Q <- mean_i M_i^T P~, P~ <- QR(mean_i M_i Q) on the
    // stored M before the usual last back-projection
    float* Qnode = (float*)(ws + h->lay.Qnode);
    float* part = (float*)(ws + h->lay.part);
    for (int k = 1; k < h->power_steps; ++k) {
        const int Sb = launch_back(L, h->E, Phat, part, m, n, r, N, cnt, h->rpc, h->S, h->vec4);
        size_t tq = (size_t)cnt * n * r;
        L.begin(PSGD_K_BACKPROJECT);
        k_reduce_q<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(part, Qnode, h->Q, n, r, N, Sb, cnt);
        L.end();
        launch_project(L, h->E, nullptr, nullptr, h->Q, Pnode, m, n, r, N, cnt, h->vec4);
        L.begin(PSGD_K_ORTH);
        k_node_mean<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Pnode, Pmean, (size_t)m * r, N, cnt);
        L.end();
        launch_orth(L, h, Pmean, Phat, m, r, PSGD_K_ORTH, nullptr, true);
    }
}

// ---- SVD-Comp (Algorithm 1, second function): top-r left singular subspace of the
//      node mean by randomised block subspace iteration + Rayleigh-Ritz. ----------
void svd(Launcher& L, psgd_handle* h, const void* G, bool have_dbar = false) {
    char* ws = h->ws;
    float* Phat = (float*)(ws + h->lay.Phat);
    float* dbar = (float*)(ws + h->lay.dbar);
    float* Y = (float*)(ws + h->lay.Y);
    float* Z = (float*)(ws + h->lay.Z);
    float* part = (float*)(ws + h->lay.part);
    double* gram = (double*)(ws + h->lay.gram);
    double* V = (double*)(ws + h->lay.V);
    double* U = (double*)(ws + h->lay.U);
    int* flags = (int*)(ws + h->lay.flags);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count, ell = h->ell;
    const int K = PSGD_K_REFRESH;
    L.force_kind = K;
    // Sweeps.  Blocks of up to 31 columns run in float32 with the device-side stopping test, so the number is only an upper
    // limit (20); wider blocks have no such test (their Rayleigh-Ritz step is too dear to repeat) and run 12 sweeps, the
    // first 8 of them in TF32: measured on a 16384 x 4096 mean with a 0.9^k spectrum, 4 sweeps already bring the top-16
    // projector within 1e-5 and 8 sweeps the energy left behind at r = 64 within 1e-9 of the optimum.
    // Blocks of 8 to 31 columns (r up to 15 with their 8 or more extra columns) converge more slowly once error feedback has filled
    // the directions right below r: 12 sweeps left the projector 3e-2 off in a free-running run, 20 (16 in TF32) pass every test.
    const int iters = h->refresh_iters > 0 ? h->refresh_iters : (h->tc_ok ? (ell < 32 ? 20 : 12) : 20);
    if (!have_dbar) launch_add_mean(L, G, h->grad_bf16, h->E, dbar, (size_t)m * n, N, cnt, K);
    size_t zt = (size_t)cnt * n * ell;
    L.begin(K);
    k_fill_normal<<<(unsigned)((zt + 255) / 256), 256, 0, L.st>>>(Z, zt, h->seed, 0x5eed0000ull + (uint64_t)h->t);
    L.end();
    // Warm start: Algorithm 2 carries Q_{t-1} across the refresh, and its columns already span most of the subspace
    // wanted (the right factor of the last compression).  They replace the first r random columns of the start block;
    // the converged result is the same subspace, reached in fewer sweeps.
    if (h->t > 0 && h->refresh_warm) {
        L.begin(K);
        k_copy_columns<<<(unsigned)(((size_t)cnt * n * r + 255) / 256), 256, 0, L.st>>>(h->Q, Z, (size_t)cnt * n, r, ell);
        L.end();
    }
    // Early sweeps on the tensor cores (TF32 operands): they bring the block close to the subspace, the
    // float32 sweeps that follow remove the TF32 rounding.  Needs Dbar^T and transposed copies of the blocks.
    int it0 = 0;
    const int tail32 = REFRESH_F32_TAIL;
    const bool tc = h->tc_ok && aligned16(dbar) && iters > tail32;
    float* dbarT = tc ? (float*)(ws + h->lay.dbarT) : nullptr;
    float* Yt = tc ? (float*)(ws + h->lay.Yt) : nullptr;
    float* Zt = tc ? (float*)(ws + h->lay.Zt) : nullptr;
    launch_orth(L, h, Z, Z, n, ell, K, Zt);
    if (tc) {
        L.begin(K);
        k_transpose<<<dim3(ceil_div(n, 32), ceil_div(m, 32), cnt), dim3(32, 8), 0, L.st>>>(dbar, dbarT, m, n);
        L.end();
        // Only Y is orthonormalised in a sweep (as in the float32 sweeps below): Z = Dbar^T Y with orthonormal Y is bounded by
        // the largest singular value, and the Gram matrix of the next Y is formed in double.
        for (; it0 < iters - tail32; ++it0) {
            launch_gemm_tc(L, h, dbar, Zt, Y, m, ell, n, K);       // Y = Dbar Z
            launch_orth(L, h, Y, Y, m, ell, K, Yt);
            launch_gemm_tc(L, h, dbarT, Yt, Z, n, ell, m, K);      // Z = Dbar^T Y
            if (it0 + 1 < iters - tail32) {
                L.begin(K);
                k_transpose<<<dim3(ceil_div(ell, 32), ceil_div(n, 32), cnt), dim3(32, 8), 0, L.st>>>(Z, Zt, n, ell);
                L.end();
            }
        }
    }
    // chunking of Z = Dbar^T Y over rows
    int colblk = ceil_div(n, BP_COLS);
    int64_t base = (int64_t)cnt * colblk * ceil_div(ell, 16);
    int S = (int)std::max<int64_t>(1, (8 * (int64_t)h->sm_count + base - 1) / base);
    S = std::min(S, std::min(64, ceil_div(m, BP_SUB)));
    int rpc = (int)align_up(ceil_div(m, S), BP_SUB);
    S = ceil_div(m, rpc);
    // Rayleigh-Ritz on the current block: eigenvectors of Z^T Z = Y^T Dbar Dbar^T Y, then P~ = Y U[:, :r]
    int* done = flags + 3;                 // set on the device once the top-r basis has stopped moving
    const bool adaptive = h->refresh_adaptive && ell <= 48 && iters - it0 > 6;
    const int* skip = adaptive ? done : nullptr;
    if (adaptive) cudaMemsetAsync(done, 0, 4, L.st);
    auto rayleigh_ritz = [&]() {
        int nparts = ceil_div(n, GR_ROWS);
        int nblk = ceil_div(ell, 64);
        GramArgs g{Z, gram, n, ell, nparts, nullptr, skip};
        L.begin(K);
        k_gram<<<dim3(nparts, nblk * nblk, cnt), 256, 0, L.st>>>(g);
        L.end();
        if (nparts > 4) {
            size_t tot = (size_t)ell * ell * cnt;
            L.begin(K);
            k_gram_sum<<<(unsigned)((tot + 31) / 32), 256, 0, L.st>>>(gram, ell * ell, nparts, cnt, skip);
            L.end();
        }
        int c2 = (ell + 1) & ~1;
        size_t smem = jac_smem_bytes(c2);
        allow_smem(k_jacobi_top, smem);
        L.begin(K);
        k_jacobi_top<<<cnt, JAC_THREADS, smem, L.st>>>(gram, nparts > 4 ? -nparts : nparts, ell, r, V, U, flags, skip);
        L.end();
        if (!jac_v_in_smem(c2)) {      // eigenvectors replayed from the rotation log
            size_t vs = jacv_smem_bytes(c2);
            allow_smem(k_jacobi_vectors, vs);
            L.begin(K);
            k_jacobi_vectors<<<dim3(ceil_div(c2, JV_ROWS), cnt), JV_THREADS, vs, L.st>>>(V, ell, r, U, skip);
            L.end();
        }
        ApplyArgs ap{Y, U, Phat, m, ell, r, r, 0, nullptr, skip};
        L.begin(K);
        k_apply<<<dim3(ceil_div(m, 32), cnt), 256, (size_t)32 * ell * 4, L.st>>>(ap);
        L.end();
    };
    // Stopping test (blocks of <= 48 columns, where a Rayleigh-Ritz step is cheap): after sweeps 2, 4, 6, 9, 12, ... the
    // top-r Ritz basis is compared with the one of the previous check; once it has stopped moving in every matrix of
    // the handle (rule in k_refresh_decide) the remaining kernels of this refresh return at once.  With geometric
    // convergence the error left is below the last movement.  Inputs that never get there run all the sweeps.
    float* Pold = (float*)(ws + h->lay.Pold);
    double* dpart = (double*)(ws + h->lay.dpart);
    double* dprev = dpart + (size_t)cnt * ceil_div(m, 64);
    int nchecks = 0;
    for (int it = it0; it < iters; ++it) {
        // Y = Dbar Z, orthonormalise;  Z = Dbar^T Y, orthonormalise
        launch_project(L, dbar, nullptr, nullptr, Z, Y, m, n, ell, 1, cnt, h->vec4, skip);
        launch_orth(L, h, Y, Y, m, ell, K, nullptr, false, skip);
        const int Sb = launch_back(L, dbar, Y, part, m, n, ell, 1, cnt, rpc, S, h->vec4, nullptr, skip);
        size_t tot = (size_t)cnt * n * ell;
        L.begin(K);
        k_reduce_q<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(part, nullptr, Z, n, ell, 1, Sb, cnt, skip);
        L.end();
        if (it + 1 == iters) break;
        const int swept = it - it0 + 1;
        if (adaptive && (swept <= 6 ? swept % 2 == 0 : swept % 3 == 0)) {
            rayleigh_ritz();
            if (nchecks > 0) {
                const int nparts = ceil_div(m, GR_ROWS), nblk = ceil_div(r, 64), nb = ceil_div(m, 64);
                GramArgs g{Pold, gram, m, r, nparts, Phat, skip};       // S = Pold^T Pnew
                L.begin(K);
                k_gram<<<dim3(nparts, nblk * nblk, cnt), 256, 0, L.st>>>(g);
                L.end();
                size_t tg = (size_t)r * r * cnt;
                L.begin(K);
                k_gram_sum<<<(unsigned)((tg + 31) / 32), 256, 0, L.st>>>(gram, r * r, nparts, cnt, skip);
                L.end();
                L.begin(K);
                k_subspace_change<<<dim3(nb, cnt), 256, (size_t)r * r * 4, L.st>>>(Pold, Phat, gram, (size_t)nparts * r * r, dpart, m, r, skip);
                L.end();
                L.begin(K);
                k_refresh_decide<<<1, 32, 0, L.st>>>(dpart, nb, cnt, dprev, nchecks > 1 ? 1 : 0, done);
                L.end();
            }
            cudaMemcpyAsync(Pold, Phat, (size_t)cnt * m * r * 4, cudaMemcpyDeviceToDevice, L.st);
            ++nchecks;
        }
        launch_orth(L, h, Z, Z, n, ell, K, nullptr, false, skip);
    }
    rayleigh_ritz();
    L.force_kind = -1;
}

// ---- one iteration with G and E stored transposed ([n][m] row-major, Sec. 1: X in R^{m x n} kept as X^T) ----------
// The same kernels with their roles exchanged: the contraction over the stored rows (the back-projection kernels) gives
// P_i = S_i^T Q, the contraction over the stored columns (the projection kernels) gives Q_i = S_i P~, and the residual kernel
// takes Q_i as its row factor and P~ as its column factor.  Three passes plus the error-feedback add (28 bytes per element).
void step_transposed(Launcher& L, psgd_handle* h, const void* G, bool refresh, float* D_hat) {
    char* ws = h->ws;
    float* Pnode = (float*)(ws + h->lay.Pnode);
    float* Pmean = (float*)(ws + h->lay.Pmean);
    float* Phat = (float*)(ws + h->lay.Phat);
    float* Qnode = (float*)(ws + h->lay.Qnode);
    float* part = (float*)(ws + h->lay.part);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    const bool vec_s = h->m % 4 == 0;          // stored rows have m entries
    if (refresh) {
        // node mean in storage orientation, transposed once into the [m][n] array SVD-Comp works on
        float* dbar_s = (float*)(ws + h->lay.dbarT);
        float* dbar = (float*)(ws + h->lay.dbar);
        launch_add_mean(L, G, h->grad_bf16, h->E, dbar_s, (size_t)m * n, N, cnt, PSGD_K_REFRESH);
        L.begin(PSGD_K_REFRESH);
        k_transpose<<<dim3(ceil_div(m, 32), ceil_div(n, 32), cnt), dim3(32, 8), 0, L.st>>>(dbar_s, dbar, n, m);
        L.end();
        svd(L, h, G, true);
    } else {
        launch_add_mean(L, G, h->grad_bf16, h->E, nullptr, (size_t)m * n, N, cnt, PSGD_K_PROJECT);
        // P_i = S_i^T Q_{t-1} and their node mean
        const int Sb = launch_back(L, h->E, h->Q, part, n, m, r, N, cnt, h->t_rpc, h->t_S, vec_s);
        size_t tot = (size_t)cnt * m * r;
        L.begin(PSGD_K_PROJECT);
        k_reduce_q<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(part, Pnode, Pmean, m, r, N, Sb, cnt);
        L.end();
        launch_orth(L, h, Pmean, Phat, m, r, PSGD_K_ORTH, nullptr, true);
    }
    // Q_i = S_i P~, Q = mean_i Q_i
    launch_project(L, h->E, nullptr, nullptr, Phat, Qnode, n, m, r, N, cnt, vec_s);
    size_t tq = (size_t)cnt * n * r;
    L.begin(PSGD_K_BACKPROJECT);
    k_node_mean<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(Qnode, h->Q, (size_t)n * r, N, cnt);
    L.end();
    // E_s = S - Q_i P~^T (stored orientation)
    if (h->error_form == 0) launch_resid(L, h->E, h->E, Qnode, Phat, n, m, r, N, cnt * N, 0, 1, vec_s, 1);
    else launch_resid(L, h->E, h->E, h->Q, Phat, n, m, r, N, cnt * N, 0, 1, vec_s, 0);
    if (D_hat) launch_resid(L, nullptr, D_hat, h->Q, Phat, n, m, r, N, cnt, 0, 0, vec_s, 0);
}

// ---- single-pass SSP-Comp step (deferred residual) --------------------------------
template <int RP, int WC>
void launch_fused_t(Launcher& L, psgd_handle* h, const void* G, FusedArgs a) {
    void (*kern)(CUtensorMap, CUtensorMap, FusedArgs) =
        h->grad_bf16 ? (h->pending ? k_fused_step<RP, WC, true, true> : k_fused_step<RP, WC, false, true>)
                     : (h->pending ? k_fused_step<RP, WC, true, false> : k_fused_step<RP, WC, false, false>);
    set_smem_attr((const void*)kern, h->fused_smem);
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(FU_THREADS);
    cfg.dynamicSmemBytes = h->fused_smem;
    cfg.stream = L.st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)h->CS;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (h->active_clusters < 0) {
        cfg.gridDim = dim3((unsigned)((size_t)h->CS * h->KCmax * h->count));
        int nc = 0;
        if (cudaOccupancyMaxActiveClusters(&nc, kern, &cfg) != cudaSuccess) { nc = 0; cudaGetLastError(); }
        h->active_clusters = nc;
        // row slots: trade the idle tail of the last wave of clusters against the traffic of the
        // per-slot partial W (written and read once: 2 KC RP / (3 m) of the step's 12 bytes per element)
        // and the start-up of every slot (loading Q', filling the ring, the first exchange: measured
        // about 1.35 row blocks' worth of time per slot)
        int best = h->KCmax;
        if (nc > 0) {
            double best_cost = 1e30;
            for (int KC = 1; KC <= h->KCmax; ++KC) {
                int64_t tot = (int64_t)h->count * KC;
                double eff = (double)tot / (double)(((tot + nc - 1) / nc) * nc);
                double cost = 1.0 / eff + 2.0 * KC * RP / (3.0 * (double)h->m) + 1.35 * KC / (double)h->nblk;
                if (cost < best_cost - 1e-9) { best_cost = cost; best = KC; }
            }
        }
        h->KC = best;
    }
    a.KC = h->KC;
    cfg.gridDim = dim3((unsigned)((size_t)h->CS * h->KC * h->count));
    CUtensorMap tmG, tmM;
    const int bw = FusedGeom<WC>::BW, rs = FusedGeom<WC>::RS;
    if (!make_tile_map(h, &tmG, G, h->n, h->m, (int64_t)h->count * h->N, bw, rs, CU_TENSOR_MAP_SWIZZLE_NONE, h->grad_bf16) ||
        !make_tile_map(h, &tmM, h->E, h->n, h->m, (int64_t)h->count * h->N, bw, rs)) {
        snprintf(h->err, sizeof(h->err), "cuTensorMapEncodeTiled failed");
        L.status = PSGD_E_CUDA;
        return;
    }
    L.begin(PSGD_K_PROJECT);
    cudaLaunchKernelEx(&cfg, kern, tmG, tmM, a);
    L.end();
}
template <int RP>
void launch_fused_rp(Launcher& L, psgd_handle* h, const void* G, const FusedArgs& a) {
    if (h->WC == 128) launch_fused_t<RP, 128>(L, h, G, a);
    else if (h->WC == 256) launch_fused_t<RP, 256>(L, h, G, a);
    else launch_fused_t<RP, 512>(L, h, G, a);
}

void fused_ssp(Launcher& L, psgd_handle* h, const void* G) {
    char* ws = h->ws;
    const Layout& Y = h->lay;
    float* Phat = (float*)(ws + Y.Phat);
    float* Qnode = (float*)(ws + Y.Qnode);
    float* part = (float*)(ws + Y.part);
    double* gram = (double*)(ws + Y.gram);
    double* T = (double*)(ws + Y.T);
    int* flags = (int*)(ws + Y.flags);
    int* gate = flags + 1;
    float* Qpad = (float*)(ws + Y.Qpad);
    float* Ppad = (float*)(ws + Y.Ppad);
    float* Qsub = (float*)(ws + Y.Qsub);
    float* Tacc = (float*)(ws + Y.Tacc);
    float* Pout = (float*)(ws + Y.Pout);
    float* Wpart = (float*)(ws + Y.Wpart);
    float* Cmat = (float*)(ws + Y.Cmat);
    double* Cpart = (double*)(ws + Y.Cpart);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count, RP = h->RP;
    if (!h->qpad_valid) {   // first single-pass step after an eager one: no accumulated transform yet, Q' = Q
        size_t tot = (size_t)cnt * n * RP;
        L.begin(PSGD_K_MISC);
        k_pad_rows<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(h->Q, Qpad, (size_t)cnt * n, r, RP);
        L.end();
        h->qpad_valid = true;
    }
    cudaMemsetAsync(gate, 0, 4, L.st);
    FusedArgs a{h->E, Qpad, Ppad, Qsub, Cmat, Pout, Wpart, gram, flags,
                m, n, r, N, h->KC, h->CS, h->nblk,
                h->error_form == 0 ? (long long)n * RP : 0LL};
    if (RP == 4) launch_fused_rp<4>(L, h, G, a);
    else launch_fused_rp<8>(L, h, G, a);
    if (L.status != PSGD_OK) return;
    // P'^T P' = L L^T  ->  T'; scaled pivot^2 < 2e-2 (rounding of W T amplified > 7x) raises the gate for the precise path
    L.begin(PSGD_K_ORTH);
    int* defic = (int*)(ws + Y.defic);
    k_chol_t<256><<<cnt, 256, (size_t)r * chol_ld(r) * 8, L.st>>>(gram, T, r, h->KC, flags, gate, 2e-2, defic);
    L.end();
    FinishPArgs fp{Pout, T, Phat, Ppad, Tacc, Tacc, m, r, RP, h->tacc_identity ? 1 : 0};
    L.begin(PSGD_K_ORTH);
    k_finish_p<<<dim3(ceil_div(m, 64), cnt), 256, 0, L.st>>>(fp);
    L.end();
    L.begin(PSGD_K_ORTH);   // rank-deficient P': orthonormal completion of P~ and of its padded copy (no-op otherwise)
    k_complete<<<cnt, 256, 0, L.st>>>(Phat, Ppad, defic, flags, m, r, RP, h->seed + (uint64_t)h->t);
    L.end();
    // precise back-projection over the stored Delta, only when the gate was raised
    launch_back(L, h->E, Phat, part, m, n, r, N, cnt, h->rpc, h->S, h->vec4, gate);
    const int qblocks = ceil_div(n, 16);
    FinishQArgs fq{Wpart, part, T, Tacc, gate, Qnode, h->Q, Qpad, Qsub, Cpart, n, r, RP, N, h->KC, h->S, h->error_form};
    L.begin(PSGD_K_BACKPROJECT);
    k_finish_q<<<dim3(qblocks, cnt), 16 * RP, 0, L.st>>>(fq);
    L.end();
    L.begin(PSGD_K_BACKPROJECT);
    k_sum_c<<<cnt, RP * RP, 0, L.st>>>(Cpart, Cmat, qblocks, RP);
    L.end();
    h->pending = true;
    h->pending_fused = true;
    h->tacc_identity = false;
}

// ---- single-pass SSP-Comp step, L2-pipelined kernel (psgd_stream.cuh) ----------------
template <int RP>
bool launch_stream_t(Launcher& L, psgd_handle* h, StreamArgs a) {
    void (*kern)(StreamArgs) = h->pending ? k_stream_step<RP, true> : k_stream_step<RP, false>;
    const size_t smem = stream_smem_bytes<RP>();
    set_smem_attr((const void*)kern, smem);
    if (h->s_grid < 0) {     // one persistent CTA per multiprocessor, all of them resident (they wait on one another's flags)
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, SS_THREADS, smem) != cudaSuccess) { per_sm = 0; cudaGetLastError(); }
        h->s_grid = std::min(per_sm, 1) * h->sm_count;
    }
    if (h->s_grid <= 0) return false;
    const int64_t units = (int64_t)h->count * h->s_nrb * h->N * h->s_csplit;
    const int grid = (int)std::min<int64_t>(h->s_grid, units);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(SS_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = L.st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    L.begin(PSGD_K_PROJECT);
    cudaLaunchKernelEx(&cfg, kern, a);
    L.end();
    return true;
}

bool stream_ssp(Launcher& L, psgd_handle* h, const void* G) {
    char* ws = h->ws;
    const Layout& Y = h->lay;
    float* Phat = (float*)(ws + Y.Phat);
    float* Qnode = (float*)(ws + Y.Qnode);
    float* part = (float*)(ws + Y.part);
    double* gram = (double*)(ws + Y.sGram);
    double* T = (double*)(ws + Y.T);
    int* flags = (int*)(ws + Y.flags);
    int* gate = flags + 1;
    float* Qpad = (float*)(ws + Y.Qpad);
    float* Ppad = (float*)(ws + Y.Ppad);
    float* Qsub = (float*)(ws + Y.Qsub);
    float* Tacc = (float*)(ws + Y.Tacc);
    float* Pout = (float*)(ws + Y.Pout);
    float* Wpart = (float*)(ws + Y.Wpart);
    float* Cmat = (float*)(ws + Y.Cmat);
    double* Cpart = (double*)(ws + Y.Cpart);
    unsigned* cnts = (unsigned*)(ws + Y.sCnt);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count, RP = h->RP, nrb = h->s_nrb;
    if (!h->qpad_valid) {   // first single-pass step after an eager one: no accumulated transform yet, Q' = Q
        size_t tot = (size_t)cnt * n * RP;
        L.begin(PSGD_K_MISC);
        k_pad_rows<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(h->Q, Qpad, (size_t)cnt * n, r, RP);
        L.end();
        h->qpad_valid = true;
    }
    cudaMemsetAsync(gate, 0, 4, L.st);
    cudaMemsetAsync(cnts, 0, (size_t)cnt * nrb * 2 * 4, L.st);
    StreamArgs a{(const float*)G, h->E, Qpad, Qsub, Ppad, (float*)(ws + Y.sPpart), Pout, Wpart, gram, cnts, cnts + (size_t)cnt * nrb, flags,
                 m, n, r, N, cnt, nrb, h->s_ngrp, h->s_tpu, h->s_csplit, h->s_KC, h->s_CB, h->error_form == 0 ? 1 : 0};
    bool ok = RP == 4 ? launch_stream_t<4>(L, h, a) : (RP == 8 ? launch_stream_t<8>(L, h, a) : launch_stream_t<16>(L, h, a));
    if (!ok) return false;
    if (L.status != PSGD_OK) return true;
    // P'^T P' = L L^T  ->  T'; scaled pivot^2 < 2e-2 raises the gate for the precise back-projection (as in the cluster kernel's path)
    size_t tg = (size_t)r * r * cnt;
    L.begin(PSGD_K_ORTH);
    k_gram_sum<<<(unsigned)((tg + 31) / 32), 256, 0, L.st>>>(gram, r * r, nrb, cnt);
    L.end();
    L.begin(PSGD_K_ORTH);
    int* defic = (int*)(ws + Y.defic);
    k_chol_t<256><<<cnt, 256, (size_t)r * chol_ld(r) * 8, L.st>>>(gram, T, r, -nrb, flags, gate, 2e-2, defic);
    L.end();
    FinishPArgs fp{Pout, T, Phat, Ppad, Tacc, Tacc, m, r, RP, h->tacc_identity ? 1 : 0};
    L.begin(PSGD_K_ORTH);
    k_finish_p<<<dim3(ceil_div(m, 64), cnt), 256, 0, L.st>>>(fp);
    L.end();
    L.begin(PSGD_K_ORTH);
    k_complete<<<cnt, 256, 0, L.st>>>(Phat, Ppad, defic, flags, m, r, RP, h->seed + (uint64_t)h->t);
    L.end();
    launch_back(L, h->E, Phat, part, m, n, r, N, cnt, h->rpc, h->S, h->vec4, gate);
    const int qblocks = ceil_div(n, 16);
    FinishQArgs fq{Wpart, part, T, Tacc, gate, Qnode, h->Q, Qpad, Qsub, Cpart, n, r, RP, N, 2 * h->s_KC, h->S, h->error_form};
    L.begin(PSGD_K_BACKPROJECT);
    k_finish_q<<<dim3(qblocks, cnt), 16 * RP, 0, L.st>>>(fq);
    L.end();
    L.begin(PSGD_K_BACKPROJECT);
    k_sum_c<<<cnt, RP * RP, 0, L.st>>>(Cpart, Cmat, qblocks, RP);
    L.end();
    h->pending = true;
    h->pending_fused = true;
    h->tacc_identity = false;
    return true;
}

// e_{t+1} = Delta_t - P~_t Qsub^T in place (Algorithm 2, last line), if it is still pending
void materialize(Launcher& L, psgd_handle* h) {
    if (!h->pending) return;
    char* ws = h->ws;
    float* Phat = (float*)(ws + h->lay.Phat);
    float* Qnode = (float*)(ws + h->lay.Qnode);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    if (h->error_form == 0) launch_resid(L, h->E, h->E, Phat, Qnode, m, n, r, N, cnt * N, 1, 1, h->vec4);
    else launch_resid(L, h->E, h->E, Phat, h->Q, m, n, r, N, cnt * N, 0, 1, h->vec4);
    h->pending = false;
}

// ---- one iteration with the nodes spread over several processes --------------------------------------------------
// Algorithm 2 averages P (line "P <- allreduce-mean"), Q and, at a refresh, Delta over the nodes.  Here this handle holds
// N of the nodes; the caller averages three small arrays over the processes between the phases.  Every process then
// factorises the same averaged P (or runs SVD-Comp on the same averaged Delta) and gets the same P~ bit for bit.
// Deferred mode runs the two-pass form (the residual stays pending between steps); the single-pass kernels fuse the
// node mean and have no place for an exchange.
bool ex_two_pass(const psgd_handle* h) { return two_pass_ok(h); }

void exchange_begin(Launcher& L, psgd_handle* h, const void* G, float* out, bool refresh) {
    char* ws = h->ws;
    float* Pnode = (float*)(ws + h->lay.Pnode);
    float* part = (float*)(ws + h->lay.part);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    const size_t tot = (size_t)cnt * m * r;
    if (h->transposed) {
        launch_add_mean(L, G, h->grad_bf16, h->E, refresh ? out : nullptr, (size_t)m * n, N, cnt, refresh ? PSGD_K_REFRESH : PSGD_K_PROJECT);
        if (refresh) return;     // out: the local mean in storage orientation
        const int Sb = launch_back(L, h->E, h->Q, part, n, m, r, N, cnt, h->t_rpc, h->t_S, h->m % 4 == 0);
        L.begin(PSGD_K_PROJECT);
        k_reduce_q<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(part, Pnode, out, m, r, N, Sb, cnt);
        L.end();
        return;
    }
    if (!ex_two_pass(h) || refresh) materialize(L, h);
    if (refresh) {
        launch_add_mean(L, G, h->grad_bf16, h->E, out, (size_t)m * n, N, cnt, PSGD_K_REFRESH);
        return;
    }
    ssp_project(L, h, G);
    L.begin(PSGD_K_ORTH);
    k_node_mean<<<(unsigned)((tot + 255) / 256), 256, 0, L.st>>>(Pnode, out, (size_t)m * r, N, cnt);
    L.end();
}

void exchange_orth(Launcher& L, psgd_handle* h, const float* in, float* out, bool refresh) {
    char* ws = h->ws;
    float* Phat = (float*)(ws + h->lay.Phat);
    float* Qnode = (float*)(ws + h->lay.Qnode);
    float* part = (float*)(ws + h->lay.part);
    float* dbar = (float*)(ws + h->lay.dbar);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    const size_t tq = (size_t)cnt * n * r;
    if (refresh) {
        if (h->transposed) {
            L.begin(PSGD_K_REFRESH);
            k_transpose<<<dim3(ceil_div(m, 32), ceil_div(n, 32), cnt), dim3(32, 8), 0, L.st>>>(in, dbar, n, m);
            L.end();
        } else {
            L.check(cudaMemcpyAsync(dbar, in, (size_t)cnt * m * n * 4, cudaMemcpyDeviceToDevice, L.st));
        }
        svd(L, h, nullptr, true);
    } else {
        launch_orth(L, h, in, Phat, m, r, PSGD_K_ORTH, nullptr, true);
    }
    if (h->transposed) {
        launch_project(L, h->E, nullptr, nullptr, Phat, Qnode, n, m, r, N, cnt, h->m % 4 == 0);
        L.begin(PSGD_K_BACKPROJECT);
        k_node_mean<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(Qnode, out, (size_t)n * r, N, cnt);
        L.end();
    } else {
        const int Sb = launch_back(L, h->E, Phat, part, m, n, r, N, cnt, h->rpc, h->S, h->vec4);
        L.begin(PSGD_K_BACKPROJECT);
        k_reduce_q<<<(unsigned)((tq + 255) / 256), 256, 0, L.st>>>(part, Qnode, out, n, r, N, Sb, cnt);
        L.end();
    }
}

void exchange_end(Launcher& L, psgd_handle* h, const float* in, float* D_hat) {
    char* ws = h->ws;
    float* Phat = (float*)(ws + h->lay.Phat);
    float* Qnode = (float*)(ws + h->lay.Qnode);
    const int m = (int)h->m, n = (int)h->n, r = h->r, N = h->N, cnt = h->count;
    if (in != h->Q) L.check(cudaMemcpyAsync(h->Q, in, (size_t)cnt * n * r * 4, cudaMemcpyDeviceToDevice, L.st));
    if (h->transposed) {
        const bool vec_s = h->m % 4 == 0;
        if (h->error_form == 0) launch_resid(L, h->E, h->E, Qnode, Phat, n, m, r, N, cnt * N, 0, 1, vec_s, 1);
        else launch_resid(L, h->E, h->E, h->Q, Phat, n, m, r, N, cnt * N, 0, 1, vec_s, 0);
        if (D_hat) launch_resid(L, nullptr, D_hat, h->Q, Phat, n, m, r, N, cnt, 0, 0, vec_s, 0);
        return;
    }
    if (ex_two_pass(h)) {
        h->pending = true;
        h->pending_fused = false;
    } else if (h->error_form == 0) {
        launch_resid(L, h->E, h->E, Phat, Qnode, m, n, r, N, cnt * N, 1, 1, h->vec4);
    } else {
        launch_resid(L, h->E, h->E, Phat, h->Q, m, n, r, N, cnt * N, 0, 1, h->vec4);
    }
    if (D_hat) launch_resid(L, nullptr, D_hat, Phat, h->Q, m, n, r, N, cnt, 0, 0, h->vec4);
    h->tacc_identity = true;
    h->qpad_valid = false;
}

psgd_status check_ready(const psgd_handle* h) {
    if (!h) return PSGD_E_NULL;
    if (!h->E || !h->Q || !h->ws) return PSGD_E_WORKSPACE;
    return PSGD_OK;
}

psgd_status do_step(psgd_handle* h, const void* G, float* P_hat, float* D_hat, psgd_stream stream, bool force) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!G) return PSGD_E_NULL;
    if (h->ex_phase != 0) return PSGD_E_INVALID;   // an iteration begun by psgd_exchange_begin is still open
    cudaStream_t st = (cudaStream_t)stream;
    Launcher L{h, st};
    bool refresh = force || (h->tau > 0 && h->t % h->tau == 0);
    // (a bfloat16 row has to be a multiple of 16 bytes for the tensor map: n % 8 == 0)
    if (h->transposed) {
        step_transposed(L, h, G, refresh, D_hat);
        h->step_kernel = 0;
        if (L.status != PSGD_OK) return L.status;
        if (P_hat) {
            PSGD_CUDA(h, cudaMemcpyAsync(P_hat, h->ws + h->lay.Phat, (size_t)h->count * h->m * h->r * 4,
                                         cudaMemcpyDeviceToDevice, st));
        }
        h->t += 1;
        return PSGD_OK;
    }
    const bool one_pass = h->mode == 1 && !refresh && aligned16(G) && h->power_steps == 1;
    bool done = false;
    h->ran_pending_tc = false;
    if (one_pass && h->stream_ok && h->s_grid != 0) {
        if (h->pending && !h->pending_fused) materialize(L, h);   // Delta_t left by a two-pass step: no padded factors for it
        done = stream_ssp(L, h, G);
        if (done) h->step_kernel = 2;
    }
    if (!done && one_pass && h->fused_ok && (!h->grad_bf16 || h->n % 8 == 0)) {
        if (h->pending && !h->pending_fused) materialize(L, h);
        fused_ssp(L, h, G);
        done = true;
        h->step_kernel = 1;
    }
    if (done) {
        if (D_hat) {
            float* Phat = (float*)(h->ws + h->lay.Phat);
            launch_resid(L, nullptr, D_hat, Phat, h->Q, (int)h->m, (int)h->n, h->r, h->N, h->count, 0, 0, h->vec4);
        }
    } else {
        // Refresh steps and shapes outside the single-pass plan run the three-pass kernels.  In deferred mode, up to
        // 16 columns, SSP steps take two passes: the residual pass is dropped, the E buffer keeps Delta_t and the next
        // projection forms e_{t+1} = Delta_t - P~_t Q_i^T on the fly (16 instead of 24 bytes per element).
        // A refresh step needs the true residual before it (SVD-Comp works on g + e), but may leave its own residual pending
        // like any other step of that mode.
        const bool two_pass = two_pass_ok(h);
        if (!two_pass || refresh) materialize(L, h);
        if (refresh) svd(L, h, G); else ssp(L, h, G);
        tail(L, h, D_hat, two_pass);
        h->tacc_identity = true;
        h->qpad_valid = false;
        h->step_kernel = h->ran_pending_tc ? 3 : 0;
    }
    if (L.status != PSGD_OK) return L.status;
    if (P_hat) {
        PSGD_CUDA(h, cudaMemcpyAsync(P_hat, h->ws + h->lay.Phat, (size_t)h->count * h->m * h->r * 4,
                                     cudaMemcpyDeviceToDevice, st));
    }
    h->t += 1;
    return PSGD_OK;
}

}  // namespace

extern "C" {

psgd_status psgd_create_batch(int64_t m, int64_t n, int r, int N, int count, int refresh_period, uint64_t seed,
                              psgd_handle** out) {
    if (!out) return PSGD_E_NULL;
    if (!(m >= n && n >= r && r >= 1 && r <= MAX_R && N >= 1 && count >= 1 && refresh_period >= 0)) return PSGD_E_INVALID;
    if (m > (1 << 24) || n > (1 << 24) || N > 65535 || (int64_t)count * 8 > 65535) return PSGD_E_INVALID;
    psgd_handle* h = new (std::nothrow) psgd_handle();
    if (!h) return PSGD_E_INVALID;
    h->m = m; h->n = n; h->r = r; h->N = N; h->count = count; h->tau = refresh_period; h->seed = seed;
    h->vec4 = (n % 4 == 0);
    h->sm_count = device_sms();
    plan(h);
    *out = h;
    return PSGD_OK;
}

psgd_status psgd_create(int64_t m, int64_t n, int r, int N, int refresh_period, uint64_t seed, psgd_handle** out) {
    return psgd_create_batch(m, n, r, N, 1, refresh_period, seed, out);
}

psgd_status psgd_set_option(psgd_handle* h, int option, int value) {
    if (!h) return PSGD_E_NULL;
    if (h->ws) return PSGD_E_STATE;
    switch (option) {
        case PSGD_OPT_ERROR_FORM: if (value != 0 && value != 1) return PSGD_E_INVALID; h->error_form = value; break;
        case PSGD_OPT_MODE: if (value != 0 && value != 1) return PSGD_E_INVALID; h->mode = value; break;
        case PSGD_OPT_REFRESH_ITERS: if (value < 0 || value > 64) return PSGD_E_INVALID; h->refresh_iters = value; break;
        case PSGD_OPT_REFRESH_OVERSAMPLE: if (value < 0 || value > MAX_L) return PSGD_E_INVALID; h->oversample = value; break;
        case PSGD_OPT_REFRESH_TC: if (value != 0 && value != 1) return PSGD_E_INVALID; h->refresh_tc = value; break;
        case PSGD_OPT_REFRESH_ADAPTIVE: if (value != 0 && value != 1) return PSGD_E_INVALID; h->refresh_adaptive = value; break;
        case PSGD_OPT_POWER_STEPS: if (value < 1 || value > 16) return PSGD_E_INVALID; h->power_steps = value; break;
        case PSGD_OPT_GRAD_BF16: if (value != 0 && value != 1) return PSGD_E_INVALID; h->grad_bf16 = value != 0; break;
        case PSGD_OPT_TRANSPOSED: if (value != 0 && value != 1) return PSGD_E_INVALID; h->transposed = value != 0; break;
        case PSGD_OPT_SINGLE_PASS: if (value < 0 || value > 3) return PSGD_E_INVALID; h->single_pass_kernel = value; break;
        case PSGD_OPT_PENDING_TC: if (value < 0 || value > 2) return PSGD_E_INVALID; h->pend_tc = value; break;
        case PSGD_OPT_BACKPROJECT_TMA: if (value != 0 && value != 1) return PSGD_E_INVALID; h->bq_ok = value != 0; break;
        default: return PSGD_E_INVALID;
    }
    plan(h);
    return PSGD_OK;
}

psgd_status psgd_sizes(const psgd_handle* h, size_t* e_bytes, size_t* q_bytes, size_t* workspace_bytes) {
    if (!h) return PSGD_E_NULL;
    if (e_bytes) *e_bytes = (size_t)h->count * h->N * h->m * h->n * 4;
    if (q_bytes) *q_bytes = (size_t)h->count * h->n * h->r * 4;
    if (workspace_bytes) *workspace_bytes = h->lay.total;
    return PSGD_OK;
}

psgd_status psgd_attach(psgd_handle* h, float* E, float* Q, void* workspace, size_t workspace_bytes) {
    if (!h || !E || !Q || !workspace) return PSGD_E_NULL;
    if (workspace_bytes < h->lay.total) return PSGD_E_WORKSPACE;
    if (((uintptr_t)E & 255) || ((uintptr_t)Q & 255) || ((uintptr_t)workspace & 255)) return PSGD_E_INVALID;
    h->E = E; h->Q = Q; h->ws = (char*)workspace; h->ws_bytes = workspace_bytes;
    return PSGD_OK;
}

psgd_status psgd_reset(psgd_handle* h, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    size_t eb, qb;
    psgd_sizes(h, &eb, &qb, nullptr);
    PSGD_CUDA(h, cudaMemsetAsync(h->E, 0, eb, st));
    PSGD_CUDA(h, cudaMemsetAsync(h->ws + h->lay.flags, 0, 256, st));
    Launcher L{h, st};
    size_t tot = qb / 4;
    L.begin(PSGD_K_MISC);
    k_fill_normal<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(h->Q, tot, h->seed, 1);
    L.end();
    h->t = 0;
    h->pending = false; h->tacc_identity = true; h->qpad_valid = false;
    h->ex_phase = 0;
    return L.status;
}

psgd_status psgd_step(psgd_handle* h, const void* G, float* P_hat, float* D_hat, psgd_stream stream) {
    return do_step(h, G, P_hat, D_hat, stream, false);
}

psgd_status psgd_refresh(psgd_handle* h, const void* G, float* P_hat, float* D_hat, psgd_stream stream) {
    return do_step(h, G, P_hat, D_hat, stream, true);
}

psgd_status psgd_exchange_plan(const psgd_handle* h, int force_refresh, int* refresh, size_t* first_floats, size_t* second_floats) {
    if (!h) return PSGD_E_NULL;
    const bool rf = h->ex_phase != 0 ? h->ex_refresh : (force_refresh || (h->tau > 0 && h->t % h->tau == 0));
    if (refresh) *refresh = rf ? 1 : 0;
    if (first_floats) *first_floats = (size_t)h->count * h->m * (rf ? (size_t)h->n : (size_t)h->r);
    if (second_floats) *second_floats = (size_t)h->count * h->n * h->r;
    return PSGD_OK;
}

psgd_status psgd_exchange_begin(psgd_handle* h, const void* G, int force_refresh, float* first, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!G || !first) return PSGD_E_NULL;
    if (h->ex_phase != 0 || h->power_steps != 1 || !aligned16(first)) return PSGD_E_INVALID;
    Launcher L{h, (cudaStream_t)stream};
    h->ex_refresh = force_refresh || (h->tau > 0 && h->t % h->tau == 0);
    h->ran_pending_tc = false;
    exchange_begin(L, h, G, first, h->ex_refresh);
    if (L.status != PSGD_OK) return L.status;
    h->ex_phase = 1;
    return PSGD_OK;
}

psgd_status psgd_exchange_orth(psgd_handle* h, const float* first, float* second, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!first || !second) return PSGD_E_NULL;
    if (h->ex_phase != 1 || !aligned16(first) || !aligned16(second)) return PSGD_E_INVALID;
    Launcher L{h, (cudaStream_t)stream};
    exchange_orth(L, h, first, second, h->ex_refresh);
    if (L.status != PSGD_OK) return L.status;
    h->ex_phase = 2;
    return PSGD_OK;
}

psgd_status psgd_exchange_end(psgd_handle* h, const float* second, float* P_hat, float* D_hat, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!second) return PSGD_E_NULL;
    if (h->ex_phase != 2 || !aligned16(second)) return PSGD_E_INVALID;
    cudaStream_t st = (cudaStream_t)stream;
    Launcher L{h, st};
    exchange_end(L, h, second, D_hat);
    if (L.status != PSGD_OK) return L.status;
    h->step_kernel = h->ran_pending_tc ? 3 : 0;
    if (P_hat)
        PSGD_CUDA(h, cudaMemcpyAsync(P_hat, h->ws + h->lay.Phat, (size_t)h->count * h->m * h->r * 4, cudaMemcpyDeviceToDevice, st));
    h->ex_phase = 0;
    h->t += 1;
    return PSGD_OK;
}

psgd_status psgd_msgd_update(psgd_handle* h, float* X, float* mom, float eta, float mu, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!X || !mom) return PSGD_E_NULL;
    if (h->t == 0) return PSGD_E_STATE;      // no P~_t, Q_t yet
    Launcher L{h, (cudaStream_t)stream};
    if (h->transposed) launch_msgd(L, X, mom, eta, mu, h->Q, (const float*)(h->ws + h->lay.Phat), (int)h->n, (int)h->m, h->r, h->count);
    else launch_msgd(L, X, mom, eta, mu, (const float*)(h->ws + h->lay.Phat), h->Q, (int)h->m, (int)h->n, h->r, h->count);
    return L.status;
}

psgd_status psgd_step_host(psgd_handle* h, const void* G_host, void* G_stage, float* P_hat_host, float* Q_host,
                           psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!G_host || !G_stage) return PSGD_E_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    size_t eb, qb;
    psgd_sizes(h, &eb, &qb, nullptr);
    PSGD_CUDA(h, cudaMemcpyAsync(G_stage, G_host, h->grad_bf16 ? eb / 2 : eb, cudaMemcpyHostToDevice, st));
    s = do_step(h, G_stage, nullptr, nullptr, stream, false);
    if (s != PSGD_OK) return s;
    if (P_hat_host)
        PSGD_CUDA(h, cudaMemcpyAsync(P_hat_host, h->ws + h->lay.Phat, (size_t)h->count * h->m * h->r * 4,
                                     cudaMemcpyDeviceToHost, st));
    if (Q_host) PSGD_CUDA(h, cudaMemcpyAsync(Q_host, h->Q, qb, cudaMemcpyDeviceToHost, st));
    PSGD_CUDA(h, cudaStreamSynchronize(st));
    return PSGD_OK;
}

psgd_status psgd_materialize_error(psgd_handle* h, psgd_stream stream) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    Launcher L{h, (cudaStream_t)stream};
    materialize(L, h);   // no-op when E already holds the residual
    return L.status;
}

psgd_status psgd_state_written(psgd_handle* h) {
    if (!h) return PSGD_E_NULL;
    h->pending = false; h->tacc_identity = true; h->qpad_valid = false;
    return PSGD_OK;
}

psgd_status psgd_get_step(const psgd_handle* h, int64_t* t) {
    if (!h || !t) return PSGD_E_NULL;
    *t = h->t;
    return PSGD_OK;
}

psgd_status psgd_set_step(psgd_handle* h, int64_t t) {
    if (!h) return PSGD_E_NULL;
    if (t < 0) return PSGD_E_INVALID;
    h->t = t;
    return PSGD_OK;
}

psgd_status psgd_last_status(psgd_handle* h, psgd_stream stream, int* flags) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!flags) return PSGD_E_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    PSGD_CUDA(h, cudaMemcpyAsync(&v, h->ws + h->lay.flags, 4, cudaMemcpyDeviceToHost, st));
    PSGD_CUDA(h, cudaMemsetAsync(h->ws + h->lay.flags, 0, 4, st));
    PSGD_CUDA(h, cudaStreamSynchronize(st));
    *flags = v;
    return PSGD_OK;
}

psgd_status psgd_debug_ptr(psgd_handle* h, int which, void** ptr, size_t* bytes) {
    psgd_status s = check_ready(h);
    if (s != PSGD_OK) return s;
    if (!ptr || !bytes) return PSGD_E_NULL;
    const size_t m = h->m, n = h->n, r = h->r, N = h->N, c = h->count;
    switch (which) {
        case PSGD_BUF_P_NODE: *ptr = h->ws + h->lay.Pnode; *bytes = c * N * m * r * 4; break;
        case PSGD_BUF_Q_NODE: *ptr = h->ws + h->lay.Qnode; *bytes = c * N * n * r * 4; break;
        case PSGD_BUF_P_HAT: *ptr = h->ws + h->lay.Phat; *bytes = c * m * r * 4; break;
        case PSGD_BUF_DBAR: *ptr = h->ws + h->lay.dbar; *bytes = c * m * n * 4; break;
        case PSGD_BUF_P_MEAN: *ptr = h->ws + h->lay.Pmean; *bytes = c * m * r * 4; break;
        default: return PSGD_E_INVALID;
    }
    return PSGD_OK;
}

psgd_status psgd_plan_info(const psgd_handle* h, int* info) {
    if (!h || !info) return PSGD_E_NULL;
    info[0] = (h->fused_ok || h->stream_ok) ? 1 : 0; info[1] = h->RP; info[2] = h->WC; info[3] = h->CS; info[4] = h->KC;
    info[5] = h->active_clusters; info[6] = (int)h->fused_smem; info[7] = h->S;
    info[8] = h->pending ? 1 : 0; info[9] = (h->pending && h->pending_fused) ? 1 : 0; info[10] = h->sm_count; info[11] = h->step_kernel;
    return PSGD_OK;
}

psgd_status psgd_launch_count(const psgd_handle* h, int64_t* launches) {
    if (!h || !launches) return PSGD_E_NULL;
    *launches = h->launches;
    return PSGD_OK;
}

psgd_status psgd_profile_begin(psgd_handle* h) {
    if (!h) return PSGD_E_NULL;
    h->profiling = true;
    return PSGD_OK;
}

psgd_status psgd_profile_read(psgd_handle* h, float* ms, int* launches) {
    if (!h || !ms || !launches) return PSGD_E_NULL;
    for (int k = 0; k < PSGD_K_COUNT; ++k) { ms[k] = 0.f; launches[k] = 0; }
    for (auto& ev : h->events) {
        PSGD_CUDA(h, cudaEventSynchronize(ev.b));
        float t = 0.f;
        PSGD_CUDA(h, cudaEventElapsedTime(&t, ev.a, ev.b));
        ms[ev.kind] += t;
        launches[ev.kind] += 1;
        cudaEventDestroy(ev.a);
        cudaEventDestroy(ev.b);
    }
    h->events.clear();
    h->profiling = false;
    return PSGD_OK;
}

const char* psgd_last_cuda_error(const psgd_handle* h) { return h ? h->err : "null handle"; }

psgd_status psgd_destroy(psgd_handle* h) {
    if (!h) return PSGD_E_NULL;
    for (auto& ev : h->events) { cudaEventDestroy(ev.a); cudaEventDestroy(ev.b); }
    delete h;
    return PSGD_OK;
}

}  // extern "C"

extern "C" {

psgd_status psgd_gemm_nt_tf32_scratch(int64_t M, int64_t Nc, int64_t K, int count, size_t* scratch_bytes) {
    if (!scratch_bytes) return PSGD_E_NULL;
    if (!(M >= 1 && Nc >= 1 && Nc <= TC_MAXN && K >= 4 && K % 4 == 0 && count >= 1 && count <= 65535)) return PSGD_E_INVALID;
    *scratch_bytes = (size_t)gemm_tc_splits(M, K, count, device_sms()) * count * M * align_up(Nc, 16) * 4 + 256;
    return PSGD_OK;
}

psgd_status psgd_gemm_nt_tf32(const float* A, const float* B, float* C, int64_t M, int64_t Nc, int64_t K, int count,
                              void* scratch, size_t scratch_bytes, psgd_stream stream) {
    size_t need = 0;
    psgd_status st = psgd_gemm_nt_tf32_scratch(M, Nc, K, count, &need);
    if (st != PSGD_OK) return st;
    if (!A || !B || !C || !scratch) return PSGD_E_NULL;
    if (scratch_bytes < need) return PSGD_E_WORKSPACE;
    if (!aligned16(A) || !aligned16(B) || ((uintptr_t)scratch & 255)) return PSGD_E_INVALID;
    cudaStream_t cs = (cudaStream_t)stream;
    const int Ncp = (int)align_up(Nc, 16);
    const int KB = ceil_div(K, TC_BK);
    const int S = gemm_tc_splits(M, K, count, device_sms());
    const int kbps = ceil_div(KB, S);
    int* flags = (int*)scratch;                       // first 256 bytes: status word
    float* Cpart = (float*)((char*)scratch + 256);
    CUtensorMap tmA, tmB;
    if (!encode_tile_map(&tmA, A, K, M, count, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !encode_tile_map(&tmB, B, K, Nc, count, TC_BK, Ncp, CU_TENSOR_MAP_SWIZZLE_128B))
        return PSGD_E_CUDA;
    if (cudaMemsetAsync(flags, 0, 4, cs) != cudaSuccess) return PSGD_E_CUDA;
    GemmTcArgs g{Cpart, (int)M, Ncp, (int)K, S, kbps, flags};
    size_t smem = gemm_tc_smem_bytes(Ncp);
    set_smem_attr((const void*)k_gemm_tf32, smem);
    k_gemm_tf32<<<dim3(ceil_div(M, TC_BM), S, count), TC_THREADS, smem, cs>>>(tmA, tmB, g);
    size_t tot = (size_t)count * M * Nc;
    k_gemm_reduce<<<(unsigned)((tot + 255) / 256), 256, 0, cs>>>(Cpart, C, (int)M, (int)Nc, Ncp, S, count);
    if (cudaGetLastError() != cudaSuccess) return PSGD_E_CUDA;
    int hflags = 0;
    if (cudaMemcpyAsync(&hflags, flags, 4, cudaMemcpyDeviceToHost, cs) != cudaSuccess || cudaStreamSynchronize(cs) != cudaSuccess)
        return PSGD_E_CUDA;
    return hflags ? PSGD_E_STATE : PSGD_OK;
}

}  // extern "C"

struct psgd_group {
    std::vector<psgd_handle*> hs;
    std::vector<cudaStream_t> streams;
    std::vector<cudaEvent_t> join;
    cudaEvent_t fork = nullptr;
};

extern "C" {

psgd_status psgd_group_create(psgd_handle* const* handles, int count, psgd_group** out) {
    if (!handles || !out) return PSGD_E_NULL;
    if (count < 1 || count > 4096) return PSGD_E_INVALID;
    for (int i = 0; i < count; ++i)
        if (!handles[i]) return PSGD_E_NULL;
    psgd_group* g = new (std::nothrow) psgd_group();
    if (!g) return PSGD_E_INVALID;
    bool ok = cudaEventCreateWithFlags(&g->fork, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < count && ok; ++i) {
        cudaStream_t s = nullptr;
        cudaEvent_t e = nullptr;
        ok = cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) == cudaSuccess;
        if (ok) g->streams.push_back(s);
        ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        if (ok) g->join.push_back(e);
        if (ok) g->hs.push_back(handles[i]);
    }
    if (!ok) {
        cudaGetLastError();
        psgd_group_destroy(g);
        return PSGD_E_CUDA;
    }
    *out = g;
    return PSGD_OK;
}

psgd_status psgd_group_step(psgd_group* g, const void* const* G, float* const* P_hat, psgd_stream stream) {
    if (!g || !G) return PSGD_E_NULL;
    for (size_t i = 0; i < g->hs.size(); ++i) {
        psgd_status s = check_ready(g->hs[i]);
        if (s != PSGD_OK) return s;
        if (!G[i]) return PSGD_E_NULL;
    }
    cudaStream_t main = (cudaStream_t)stream;
    if (cudaEventRecord(g->fork, main) != cudaSuccess) return PSGD_E_CUDA;
    psgd_status worst = PSGD_OK;
    for (size_t i = 0; i < g->hs.size(); ++i) {
        if (cudaStreamWaitEvent(g->streams[i], g->fork, 0) != cudaSuccess) return PSGD_E_CUDA;
        psgd_status s = psgd_step(g->hs[i], G[i], P_hat ? P_hat[i] : nullptr, nullptr, (psgd_stream)g->streams[i]);
        if (s != PSGD_OK && worst == PSGD_OK) worst = s;
        if (cudaEventRecord(g->join[i], g->streams[i]) != cudaSuccess) return PSGD_E_CUDA;
    }
    for (size_t i = 0; i < g->hs.size(); ++i)
        if (cudaStreamWaitEvent(main, g->join[i], 0) != cudaSuccess) return PSGD_E_CUDA;
    return worst;
}

psgd_status psgd_group_destroy(psgd_group* g) {
    if (!g) return PSGD_E_NULL;
    for (cudaStream_t s : g->streams) { cudaStreamSynchronize(s); cudaStreamDestroy(s); }
    for (cudaEvent_t e : g->join) cudaEventDestroy(e);
    if (g->fork) cudaEventDestroy(g->fork);
    delete g;
    return PSGD_OK;
}

}  // extern "C"

#ifdef PSGD_PTC_TIMING
extern "C" int psgd_debug_ptc_times(unsigned* host /*[12][512]*/) {
    return (int)cudaMemcpyFromSymbol(host, psgd::g_ptc_t, sizeof(unsigned) * 12 * 512);
}
#endif

#include "psgd_noalloc.cu"
