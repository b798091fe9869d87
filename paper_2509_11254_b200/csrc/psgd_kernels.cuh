// Device kernels of the PowerSGD+ compression path (sm_100a).
//
// Naming follows the paper: M (= Delta) is g + e (Eq. (7a)); P = M Q, P~ = QR(P),
// Q_i = M_i^T P~ (Algorithm 1); e <- M - P~ Q_i^T (Algorithm 2, last line).
// All streaming kernels are HBM-bound fp32 FFMA kernels: they move tiles with
// 128-bit cp.async / 128-bit loads and keep the small factors (Q, P~) in shared
// memory where one warp reads them as broadcasts.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace psgd {

// ----------------------------------------------------------------------------
// small helpers
// ----------------------------------------------------------------------------
__device__ __forceinline__ void cp_async16(void* smem, const void* gmem, int src_bytes) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async4(void* smem, const void* gmem, int src_bytes) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ float4 ldg_stream4(const float* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}

// Two packed floats in one 64-bit register (low half = .x), kept packed from the load to the last use so
// that no pack / unpack moves are needed around the packed FMA.
typedef unsigned long long f2p;
__device__ __forceinline__ f2p pack2(float x, float y) {
    f2p d;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(d) : "f"(x), "f"(y));
    return d;
}
__device__ __forceinline__ float2 unpack2(f2p v) {
    float2 d;
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(d.x), "=f"(d.y) : "l"(v));
    return d;
}
// d = a * b + c on two packed floats (one instruction slot on sm_100)
__device__ __forceinline__ f2p ffma2(f2p a, f2p b, f2p c) {
    f2p d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// ----------------------------------------------------------------------------
// K1  project:  P_i = (A_i [+ B_i]) Q      (Algorithm 1: P^(i) <- Delta^(i) Q, with
//     the error-feedback add of Eq. (7a) fused in; optionally stores M = A + B).
//
// One CTA owns 32 rows of one (matrix, node) and walks the n columns in tiles of
// PJ_TC.  A tile is staged in shared memory by cp.async (3 stages); lane = row,
// warp = 8-column slice, so the Q tile is read as a warp-wide broadcast and each
// thread keeps RP running sums.  The 8 warps' partial sums are added in a fixed
// order at the end (deterministic).
// ----------------------------------------------------------------------------
constexpr int PJ_TR = 32;          // rows per CTA
constexpr int PJ_TC = 64;          // columns per tile
constexpr int PJ_TCP = PJ_TC + 4;  // padded row stride (floats): conflict-free 128-bit row reads
constexpr int PJ_STAGES = 3;
constexpr int PJ_THREADS = 256;

struct ProjectArgs {
    const float* A;   // [mats][rows][n]
    const float* B;   // [mats][rows][n] or nullptr
    float* Mout;      // [mats][rows][n] or nullptr (may alias B)
    const float* Q;   // [count][n][r]
    float* P;         // [mats][rows][r]
    int rows, n, r, nodes, nchunks;
    const int* skip;  // when non-null the kernel does nothing if *skip != 0 (refresh already converged)
    // PEND only (two-pass deferred mode): B holds Delta_{t-1}; the residual e_t = Delta_{t-1} - P~_{t-1} Qsub^T
    // (Algorithm 2, last line) is formed on the fly from the small factors instead of being read
    const float* Pprev = nullptr;   // [count][rows][r]
    const float* Qsub = nullptr;    // [mats][n][r] (qsub_per_node) or [count][n][r]
    int qsub_per_node = 0;
};

template <int RP, bool ADD, bool PEND = false>
__host__ __device__ constexpr size_t project_smem_bytes() {
    size_t tiles = (size_t)PJ_STAGES * PJ_TR * PJ_TCP * (ADD ? 2 : 1);
    size_t q = (size_t)PJ_STAGES * PJ_TC * RP * (PEND ? 2 : 1);
    size_t red = (size_t)8 * 32 * RP;
    size_t body = tiles + q;
    return 4 * (body > red ? body : red);
}

template <int RP, int VEC, bool ADD, bool STORE, bool PEND = false>
__global__ void __launch_bounds__(PJ_THREADS) k_project(ProjectArgs a) {
    extern __shared__ __align__(16) float smem[];
    if (a.skip && *a.skip) return;
    float* tA = smem;
    float* tB = tA + (ADD ? PJ_STAGES * PJ_TR * PJ_TCP : 0);
    float* tQ = tB + PJ_STAGES * PJ_TR * PJ_TCP;
    float* tQs = tQ + PJ_STAGES * PJ_TC * RP;      // PEND: tiles of Qsub beside those of Q

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int row0 = blockIdx.x * PJ_TR;
    const int node = blockIdx.y;
    const int c = blockIdx.z / a.nchunks, chunk = blockIdx.z % a.nchunks;
    const int k0 = chunk * RP;
    const size_t mat = (size_t)c * a.nodes + node;
    const float* Ab = a.A + mat * (size_t)a.rows * a.n;
    const float* Bb = ADD ? a.B + mat * (size_t)a.rows * a.n : nullptr;
    float* Mb = STORE ? a.Mout + mat * (size_t)a.rows * a.n : nullptr;
    const float* Qb = a.Q + (size_t)c * a.n * a.r;
    const float* Qsb = PEND ? a.Qsub + (a.qsub_per_node ? mat : (size_t)c) * a.n * a.r : nullptr;
    const int n = a.n, r = a.r, rows = a.rows;
    const int ntiles = (n + PJ_TC - 1) / PJ_TC;

    auto load_tile = [&](int t, int stage) {
        const int col0 = t * PJ_TC;
        float* sa = tA + stage * PJ_TR * PJ_TCP;
        float* sb = tB + stage * PJ_TR * PJ_TCP;
        if (VEC == 4) {
#pragma unroll
            for (int it = 0; it < (PJ_TR * PJ_TC / 4) / PJ_THREADS; ++it) {
                int ch = tid + it * PJ_THREADS;
                int rr = ch / (PJ_TC / 4), c4 = (ch % (PJ_TC / 4)) * 4;
                int grow = min(row0 + rr, rows - 1);
                int gcol = col0 + c4;
                int ok = gcol < n ? 16 : 0;
                size_t off = (size_t)grow * n + (ok ? gcol : 0);
                cp_async16(sa + rr * PJ_TCP + c4, Ab + off, ok);
                if (ADD) cp_async16(sb + rr * PJ_TCP + c4, Bb + off, ok);
            }
        } else {
            for (int e = tid; e < PJ_TR * PJ_TC; e += PJ_THREADS) {
                int rr = e / PJ_TC, cc = e % PJ_TC;
                int grow = min(row0 + rr, rows - 1);
                int gcol = col0 + cc;
                int ok = gcol < n ? 4 : 0;
                size_t off = (size_t)grow * n + (ok ? gcol : 0);
                cp_async4(sa + rr * PJ_TCP + cc, Ab + off, ok);
                if (ADD) cp_async4(sb + rr * PJ_TCP + cc, Bb + off, ok);
            }
        }
        float* sq = tQ + stage * PJ_TC * RP;
        for (int e = tid; e < PJ_TC * RP; e += PJ_THREADS) {
            int cc = e / RP, k = e % RP;
            int gcol = col0 + cc;
            int ok = (gcol < n && k0 + k < r) ? 4 : 0;
            size_t off = ok ? (size_t)gcol * r + k0 + k : 0;
            cp_async4(sq + e, Qb + off, ok);
            // Qsub tile with adjacent columns interleaved: {qs[2c][k], qs[2c+1][k]} is one 64-bit operand of the packed FMA
            if (PEND) cp_async4(tQs + stage * PJ_TC * RP + ((cc >> 1) * RP + k) * 2 + (cc & 1), Qsb + off, ok);
        }
    };
    f2p pp[PEND ? RP : 1];            // PEND: this lane's row of P~_{t-1}, every value twice (one per column of a pair)
    if (PEND) {
#pragma unroll
        for (int k = 0; k < RP; ++k) {
            const float pv = (row0 + lane < rows && k0 + k < r) ? __ldg(a.Pprev + ((size_t)c * rows + row0 + lane) * r + k0 + k) : 0.f;
            pp[k] = pack2(pv, pv);
        }
    }
    f2p acc2[PEND ? RP / 2 : 1];      // PEND: the running sums packed in pairs of adjacent k (the kernel is FMA-bound then)
#pragma unroll
    for (int k = 0; k < (PEND ? RP / 2 : 1); ++k) acc2[k] = 0ull;

    float acc[RP];
#pragma unroll
    for (int k = 0; k < RP; ++k) acc[k] = 0.f;

    for (int s = 0; s < PJ_STAGES - 1; ++s) {
        if (s < ntiles) load_tile(s, s);
        cp_async_commit();
    }
    for (int t = 0; t < ntiles; ++t) {
        cp_async_wait<PJ_STAGES - 2>();
        __syncthreads();
        if (t + PJ_STAGES - 1 < ntiles) load_tile(t + PJ_STAGES - 1, (t + PJ_STAGES - 1) % PJ_STAGES);
        cp_async_commit();
        const int stage = t % PJ_STAGES;
        float* sa = tA + stage * PJ_TR * PJ_TCP + lane * PJ_TCP;
        const float* sb = tB + stage * PJ_TR * PJ_TCP + lane * PJ_TCP;
        const float* sq = tQ + stage * PJ_TC * RP;
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int cb = warp * 8 + j * 4;
            float4 v = *reinterpret_cast<const float4*>(sa + cb);
            if (ADD) {
                float4 w = *reinterpret_cast<const float4*>(sb + cb);
                if constexpr (PEND) {     // e = Delta_{t-1} - P~_{t-1} Qsub^T for the 4 columns, k ascending as in k_residual
                    f2p corr2[2] = {0ull, 0ull};   // columns (0, 1) and (2, 3)
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {
                        const ulonglong2* qs = reinterpret_cast<const ulonglong2*>(tQs + stage * PJ_TC * RP + ((cb >> 1) + c2) * RP * 2);
#pragma unroll
                        for (int k2 = 0; k2 < RP / 2; ++k2) {
                            const ulonglong2 q2 = qs[k2];      // column pair at k = 2 k2 and 2 k2 + 1
                            corr2[c2] = ffma2(pp[2 * k2 + 0], q2.x, corr2[c2]);
                            corr2[c2] = ffma2(pp[2 * k2 + 1], q2.y, corr2[c2]);
                        }
                    }
                    const float2 c01 = unpack2(corr2[0]), c23 = unpack2(corr2[1]);
                    w.x -= c01.x; w.y -= c01.y; w.z -= c23.x; w.w -= c23.y;
                }
                v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
            }
            if (STORE) *reinterpret_cast<float4*>(sa + cb) = v;
            const float mv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) {
                const float* q = sq + (cb + cc) * RP;
                if constexpr (PEND) {
                    const f2p md = pack2(mv[cc], mv[cc]);
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const ulonglong2 qv = *reinterpret_cast<const ulonglong2*>(q + 4 * k4);
                        acc2[2 * k4 + 0] = ffma2(md, qv.x, acc2[2 * k4 + 0]);
                        acc2[2 * k4 + 1] = ffma2(md, qv.y, acc2[2 * k4 + 1]);
                    }
                    continue;
                }
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    float4 qv = *reinterpret_cast<const float4*>(q + 4 * k4);
                    acc[4 * k4 + 0] = fmaf(mv[cc], qv.x, acc[4 * k4 + 0]);
                    acc[4 * k4 + 1] = fmaf(mv[cc], qv.y, acc[4 * k4 + 1]);
                    acc[4 * k4 + 2] = fmaf(mv[cc], qv.z, acc[4 * k4 + 2]);
                    acc[4 * k4 + 3] = fmaf(mv[cc], qv.w, acc[4 * k4 + 3]);
                }
            }
        }
        if (STORE) {
            __syncthreads();
            const int col0 = t * PJ_TC;
            const float* st = tA + stage * PJ_TR * PJ_TCP;
            if (VEC == 4) {
#pragma unroll
                for (int it = 0; it < (PJ_TR * PJ_TC / 4) / PJ_THREADS; ++it) {
                    int ch = tid + it * PJ_THREADS;
                    int rr = ch / (PJ_TC / 4), c4 = (ch % (PJ_TC / 4)) * 4;
                    if (row0 + rr < rows && col0 + c4 < n)
                        *reinterpret_cast<float4*>(Mb + (size_t)(row0 + rr) * n + col0 + c4) =
                            *reinterpret_cast<const float4*>(st + rr * PJ_TCP + c4);
                }
            } else {
                for (int e = tid; e < PJ_TR * PJ_TC; e += PJ_THREADS) {
                    int rr = e / PJ_TC, cc = e % PJ_TC;
                    if (row0 + rr < rows && col0 + cc < n)
                        Mb[(size_t)(row0 + rr) * n + col0 + cc] = st[rr * PJ_TCP + cc];
                }
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();
    if constexpr (PEND) {
#pragma unroll
        for (int k = 0; k < RP / 2; ++k) {
            const float2 t2 = unpack2(acc2[k]);
            acc[2 * k] = t2.x;
            acc[2 * k + 1] = t2.y;
        }
    }
    // cross-warp reduction, fixed order
    float* red = smem;  // [8][32][RP]
#pragma unroll
    for (int k = 0; k < RP; ++k) red[(warp * 32 + lane) * RP + k] = acc[k];
    __syncthreads();
    float* Pb = a.P + mat * (size_t)rows * r;
    for (int e = tid; e < 32 * RP; e += PJ_THREADS) {
        int rr = e / RP, k = e % RP;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) s += red[(w * 32 + rr) * RP + k];
        if (row0 + rr < rows && k0 + k < r) Pb[(size_t)(row0 + rr) * r + k0 + k] = s;
    }
}

// ----------------------------------------------------------------------------
// K3  back-project:  partial Q_i = M_i[rows of chunk]^T P~   (Algorithm 1:
//     Q^(i) <- Delta^(i)^T P~).  Thread owns 4 adjacent columns and RP outputs per
//     column; P~ rows are broadcast from shared memory.  Row chunks write partial
//     sums that k_reduce_q adds in a fixed order.
// ----------------------------------------------------------------------------
constexpr int BP_THREADS = 128;
constexpr int BP_COLS = 256;   // columns per CTA (64 threads x 4)
constexpr int BP_SUB = 64;     // rows per shared-memory sub-tile of P~

struct BackArgs {
    const float* M;     // [mats][rows][n]
    const float* Phat;  // [count][rows][r]
    float* part;        // [mats][S][n][r]
    int rows, n, r, nodes, nchunks, rows_per_chunk, S;
    const int* gate;    // when non-null the kernel does nothing unless *gate != 0
    const int* skip;    // when non-null the kernel does nothing if *skip != 0
};

template <int RP, int VEC>
__global__ void __launch_bounds__(BP_THREADS) k_backproject(BackArgs a) {
    __shared__ __align__(16) float Ps[BP_SUB * RP];
    __shared__ __align__(16) float red[64 * 4 * RP];
    if (a.gate && *a.gate == 0) return;
    if (a.skip && *a.skip) return;
    const int tid = threadIdx.x, tx = tid & 63, g = tid >> 6;
    const int col = blockIdx.x * BP_COLS + tx * 4;
    const int s = blockIdx.y;
    const int mat = blockIdx.z / a.nchunks, chunk = blockIdx.z % a.nchunks;
    const int c = mat / a.nodes;
    const int k0 = chunk * RP;
    const int n = a.n, r = a.r;
    const int rbeg = s * a.rows_per_chunk, rend = min(a.rows, rbeg + a.rows_per_chunk);
    const float* Mb = a.M + (size_t)mat * a.rows * n;
    const float* Pb = a.Phat + (size_t)c * a.rows * r;

    // The sums are kept packed in pairs of adjacent k (fma.rn.f32x2: half the FMA issue slots; measured 15-25 % faster up
    // to 8 columns, 7 % at 16).
    constexpr bool PACKED = RP <= 16;
    float acc[4][RP];
    f2p acc2[4][PACKED ? RP / 2 : 1];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int k = 0; k < RP; ++k) acc[j][k] = 0.f;
#pragma unroll
        for (int k = 0; k < (PACKED ? RP / 2 : 1); ++k) acc2[j][k] = 0ull;
    }

    auto load8 = [&](int sub0, int rr, float4 (&dst)[8]) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int grow = sub0 + g + 2 * (rr + u);
            dst[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (grow < rend) {
                const float* p = Mb + (size_t)grow * n + col;
                if (VEC == 4) {
                    if (col < n) dst[u] = ldg_stream4(p);
                } else {
                    if (col + 0 < n) dst[u].x = __ldcs(p + 0);
                    if (col + 1 < n) dst[u].y = __ldcs(p + 1);
                    if (col + 2 < n) dst[u].z = __ldcs(p + 2);
                    if (col + 3 < n) dst[u].w = __ldcs(p + 3);
                }
            }
        }
    };
    float4 vn[8];
    load8(rbeg, 0, vn);
    for (int sub0 = rbeg; sub0 < rend; sub0 += BP_SUB) {
        __syncthreads();
        for (int e = tid; e < BP_SUB * RP; e += BP_THREADS) {
            int rr = e / RP, k = e % RP;
            int grow = sub0 + rr;
            Ps[e] = (grow < rend && k0 + k < r) ? Pb[(size_t)grow * r + k0 + k] : 0.f;
        }
        __syncthreads();
#pragma unroll 1
        for (int rr = 0; rr < BP_SUB / 2; rr += 8) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = vn[u];
            // the next 8 rows (of this sub-tile, else of the next one) are requested before these are used
            if (rr + 8 < BP_SUB / 2) load8(sub0, rr + 8, vn); else load8(sub0 + BP_SUB, 0, vn);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float* pr = Ps + (g + 2 * (rr + u)) * RP;
                if constexpr (PACKED) {
                    const f2p vd[4] = {pack2(v[u].x, v[u].x), pack2(v[u].y, v[u].y), pack2(v[u].z, v[u].z), pack2(v[u].w, v[u].w)};
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const ulonglong2 p4 = *reinterpret_cast<const ulonglong2*>(pr + 4 * k4);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            acc2[j][(2 * k4 + 0)] = ffma2(vd[j], p4.x, acc2[j][(2 * k4 + 0)]);
                            acc2[j][(2 * k4 + 1)] = ffma2(vd[j], p4.y, acc2[j][(2 * k4 + 1)]);
                        }
                    }
                } else {
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    float4 p4 = *reinterpret_cast<const float4*>(pr + 4 * k4);
                    const float pk[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        acc[0][4 * k4 + kk] = fmaf(v[u].x, pk[kk], acc[0][4 * k4 + kk]);
                        acc[1][4 * k4 + kk] = fmaf(v[u].y, pk[kk], acc[1][4 * k4 + kk]);
                        acc[2][4 * k4 + kk] = fmaf(v[u].z, pk[kk], acc[2][4 * k4 + kk]);
                        acc[3][4 * k4 + kk] = fmaf(v[u].w, pk[kk], acc[3][4 * k4 + kk]);
                    }
                }
                }
            }
        }
    }
    if constexpr (PACKED) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < RP; k += 2) {
                const float2 t2 = unpack2(acc2[j][(k >> 1)]);
                acc[j][k] = t2.x;
                acc[j][k + 1] = t2.y;
            }
    }
    __syncthreads();
    if (g == 1) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < RP; ++k) red[(tx * 4 + j) * RP + k] = acc[j][k];
    }
    __syncthreads();
    if (g == 0) {
        float* out = a.part + ((size_t)mat * a.S + s) * (size_t)n * r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (col + j < n) {
#pragma unroll
                for (int k = 0; k < RP; ++k)
                    if (k0 + k < r) out[(size_t)(col + j) * r + k0 + k] = acc[j][k] + red[(tx * 4 + j) * RP + k];
            }
        }
    }
}

// Q_i = sum over row chunks of the partials;  Q = (1/N) sum_i Q_i   (All-Reduce Mean).
// One thread per (matrix, column, k); fixed summation order.
__global__ void k_reduce_q(const float* part, float* Qi, float* Qmean, int n, int r, int nodes, int S, int count,
                           const int* skip = nullptr) {
    if (skip && *skip) return;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t per = (size_t)n * r;
    if (idx >= per * count) return;
    int c = (int)(idx / per);
    size_t e = idx % per;
    float tot = 0.f;
    for (int i = 0; i < nodes; ++i) {
        size_t mat = (size_t)c * nodes + i;
        float s = 0.f;
        for (int k = 0; k < S; ++k) s += part[(mat * S + k) * per + e];
        if (Qi) Qi[mat * per + e] = s;
        tot += s;
    }
    Qmean[(size_t)c * per + e] = tot / (float)nodes;
}

// ----------------------------------------------------------------------------
// K4  residual:  E_i = M_i - P~ Q_i^T   (Algorithm 2, last line), or with M == nullptr
//     the dense reconstruction P~ Q^T (Algorithm 1, return value).  Thread owns 4
//     adjacent columns with their Q rows in registers and walks the rows.
// ----------------------------------------------------------------------------
constexpr int RS_THREADS = 128;
constexpr int RS_COLS = 256;
constexpr int RS_SUB = 16;  // rows per sub-tile (8 per row group)
constexpr int RS_MAXR = 128;

struct ResidArgs {
    const float* M;     // [mats][rows][n] or nullptr
    float* Out;         // [mats][rows][n] (may alias M)
    const float* Phat;  // [count][rows][r]
    const float* Qf;    // [mats or count][n][r]
    int rows, n, r, nodes, rows_per_chunk;
    int q_per_node;     // 1: Qf indexed by (matrix,node); 0: by matrix only
    int out_per_node;   // 1: Out/M indexed by (matrix,node); 0: by matrix only (dense reconstruction)
    int p_per_node = 0; // 1: Phat (the row factor) indexed by (matrix,node); 0: by matrix only
    // momentum-SGD hand-off (Eq. (7c)), only with M == nullptr: instead of storing the reconstruction D^,
    // mom <- mu mom + D^ and X <- X - eta mom, both [mats][rows][n]
    float* X = nullptr;
    float* Mom = nullptr;
    float eta = 0.f, mu = 0.f;
};

template <int RP, int VEC>
__global__ void __launch_bounds__(RS_THREADS) k_residual(ResidArgs a) {
    __shared__ __align__(16) float Ps[RS_SUB * RS_MAXR];
    const int tid = threadIdx.x, tx = tid & 63, g = tid >> 6;
    const int col = blockIdx.x * RS_COLS + tx * 4;
    const int n = a.n, r = a.r;
    const int mat = blockIdx.z;
    const int c = a.out_per_node ? mat / a.nodes : mat;
    const int rbeg = blockIdx.y * a.rows_per_chunk, rend = min(a.rows, rbeg + a.rows_per_chunk);
    const float* Mb = a.M ? a.M + (size_t)mat * a.rows * n : nullptr;
    float* Ob = a.X ? a.X + (size_t)mat * a.rows * n : a.Out + (size_t)mat * a.rows * n;
    float* Vb = a.X ? a.Mom + (size_t)mat * a.rows * n : nullptr;
    const float* Pb = a.Phat + (size_t)(a.p_per_node ? mat : c) * a.rows * r;
    const float* Qb = a.Qf + (size_t)(a.q_per_node ? mat : c) * n * r;
    const int nch = (r + RP - 1) / RP;
    const int rpad = nch * RP;

    float q[4][RP];
    auto load_q = [&](int k0) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < RP; ++k)
                q[j][k] = (col + j < n && k0 + k < r) ? __ldg(Qb + (size_t)(col + j) * r + k0 + k) : 0.f;
    };
    if (nch == 1) load_q(0);

    for (int sub0 = rbeg; sub0 < rend; sub0 += RS_SUB) {
        __syncthreads();
        for (int e = tid; e < RS_SUB * rpad; e += RS_THREADS) {
            int rr = e / rpad, k = e % rpad;
            int grow = sub0 + rr;
            Ps[rr * RS_MAXR + k] = (grow < rend && k < r) ? Pb[(size_t)grow * r + k] : 0.f;
        }
        __syncthreads();
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int grow = sub0 + g + 2 * u;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (Mb && grow < rend) {
                const float* p = Mb + (size_t)grow * n + col;
                if (VEC == 4) {
                    if (col < n) v[u] = ldg_stream4(p);
                } else {
                    if (col + 0 < n) v[u].x = __ldcs(p + 0);
                    if (col + 1 < n) v[u].y = __ldcs(p + 1);
                    if (col + 2 < n) v[u].z = __ldcs(p + 2);
                    if (col + 3 < n) v[u].w = __ldcs(p + 3);
                }
            }
        }
        float rec[8][4];
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int j = 0; j < 4; ++j) rec[u][j] = 0.f;
        for (int ch = 0; ch < nch; ++ch) {
            if (nch > 1) load_q(ch * RP);
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float* pr = Ps + (g + 2 * u) * RS_MAXR + ch * RP;
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    float4 p4 = *reinterpret_cast<const float4*>(pr + 4 * k4);
                    const float pk[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                        for (int j = 0; j < 4; ++j) rec[u][j] = fmaf(pk[kk], q[j][4 * k4 + kk], rec[u][j]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            int grow = sub0 + g + 2 * u;
            if (grow >= rend) continue;
            float4 o;
            if (Mb) {
                o = make_float4(v[u].x - rec[u][0], v[u].y - rec[u][1], v[u].z - rec[u][2], v[u].w - rec[u][3]);
            } else {
                o = make_float4(rec[u][0], rec[u][1], rec[u][2], rec[u][3]);
            }
            float* p = Ob + (size_t)grow * n + col;
            if (Vb) {               // o is the reconstruction D^ here
                float* pv = Vb + (size_t)grow * n + col;
                const float d[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (col + j < n) {
                        const float mnew = fmaf(a.mu, pv[j], d[j]);
                        pv[j] = mnew;
                        p[j] = fmaf(-a.eta, mnew, p[j]);
                    }
                }
                continue;
            }
            if (VEC == 4) {
                if (col < n) *reinterpret_cast<float4*>(p) = o;
            } else {
                if (col + 0 < n) p[0] = o.x;
                if (col + 1 < n) p[1] = o.y;
                if (col + 2 < n) p[2] = o.z;
                if (col + 3 < n) p[3] = o.w;
            }
        }
    }
}

// ----------------------------------------------------------------------------
// elementwise helpers
// ----------------------------------------------------------------------------
// M = G + E (Eq. (7a)) written over E; optionally Dbar = (1/N) sum_i M_i (SVD-Comp, first line).
// float32 value of a gradient element: float32 as stored, bfloat16 widened exactly (its 16 bits are the top half)
__device__ __forceinline__ float grad_value(const float* G, size_t i) { return __ldcs(G + i); }
__device__ __forceinline__ float grad_value(const unsigned short* G, size_t i) { return __uint_as_float((unsigned)__ldcs(G + i) << 16); }

__device__ __forceinline__ float4 grad_value4(const float* G, size_t i) { return __ldcs(reinterpret_cast<const float4*>(G + i)); }
__device__ __forceinline__ float4 grad_value4(const unsigned short* G, size_t i) {
    const uint2 b = __ldcs(reinterpret_cast<const uint2*>(G + i));
    return make_float4(__uint_as_float(b.x << 16), __uint_as_float(b.x & 0xFFFF0000u), __uint_as_float(b.y << 16), __uint_as_float(b.y & 0xFFFF0000u));
}

// VEC == 4: per_mat % 4 == 0 and all three arrays 16-byte aligned (8-byte for bfloat16 G); a thread owns 4 adjacent
// elements of one matrix for all its nodes (128-bit accesses, the matrix index comes from blockIdx.y: no division).
// grid: (x: any, y: count).
template <typename TG, int VEC>
__global__ void __launch_bounds__(256) k_add_mean(const TG* G, float* E, float* Dbar, size_t per_mat, int nodes, int count) {
    const size_t c = blockIdx.y;
    const float nf = (float)nodes;
    const size_t stride = (size_t)gridDim.x * blockDim.x * VEC;
    for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * VEC; e < per_mat; e += stride) {
        if (VEC == 4) {
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int i = 0; i < nodes; ++i) {
                const size_t off = (c * nodes + i) * per_mat + e;
                const float4 g = grad_value4(G, off);
                float4 m = *reinterpret_cast<const float4*>(E + off);
                m.x += g.x; m.y += g.y; m.z += g.z; m.w += g.w;
                *reinterpret_cast<float4*>(E + off) = m;
                s.x += m.x; s.y += m.y; s.z += m.z; s.w += m.w;
            }
            if (Dbar) *reinterpret_cast<float4*>(Dbar + c * per_mat + e) = make_float4(s.x / nf, s.y / nf, s.z / nf, s.w / nf);
        } else {
            float s = 0.f;
            for (int i = 0; i < nodes; ++i) {
                const size_t off = (c * nodes + i) * per_mat + e;
                const float mval = grad_value(G, off) + E[off];
                E[off] = mval;
                s += mval;
            }
            if (Dbar) Dbar[c * per_mat + e] = s / nf;
        }
    }
}

// Dst[row][k] = Src[row][k] for k < c_src: the first columns of a wider row-major block.  One thread per source entry.
__global__ void k_copy_columns(const float* Src, float* Dst, size_t rows, int c_src, int c_dst) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * c_src) return;
    size_t row = idx / c_src;
    int k = (int)(idx % c_src);
    Dst[row * c_dst + k] = Src[idx];
}

// X = (1/N) sum_i X_i  for the small factor arrays (All-Reduce Mean of P).
__global__ void k_node_mean(const float* Xi, float* X, size_t per_mat, int nodes, int count) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= per_mat * count) return;
    size_t c = idx / per_mat, e = idx % per_mat;
    float s = 0.f;
    for (int i = 0; i < nodes; ++i) s += Xi[(c * nodes + i) * per_mat + e];
    X[idx] = s / (float)nodes;
}

// Counter-based N(0,1): splitmix64 of (seed, stream, index) -> two uniforms -> Box-Muller.
__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
    x += 0x9E3779B97F4A7C15ull;
    x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
    x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}
__global__ void k_fill_normal(float* X, size_t count, uint64_t seed, uint64_t stream) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= count) return;
    uint64_t h = splitmix64(splitmix64(seed ^ (stream * 0xD1B54A32D192ED03ull)) + idx);
    float u1 = ((float)(uint32_t)(h >> 40) + 0.5f) * (1.0f / 16777216.0f);
    float u2 = ((float)(uint32_t)((h >> 8) & 0xFFFFFF) + 0.5f) * (1.0f / 16777216.0f);
    X[idx] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
}

// ----------------------------------------------------------------------------
// K2  orthogonalisation  P~ = QR(P)  with diag(R) > 0, as column-scaled Cholesky QR:
//     G = P^T P (double),  d = sqrt(diag G),  D^-1 G D^-1 = L L^T,  P~ = P D^-1 L^-T.
//     For full column rank this is the unique QR factor with positive diagonal
//     (R = L^T D), i.e. what Householder QR with the sign fix returns.
// ----------------------------------------------------------------------------
constexpr int GR_ROWS = 128;  // rows per Gram CTA
struct GramArgs {
    const float* X;  // [count][rows][c]
    double* part;    // [count][nparts][c][c]
    int rows, c, nparts;
    const float* X2; // optional second factor: part = X^T X2 (all blocks computed); nullptr: X^T X, upper block triangle
    const int* skip; // when non-null the kernel does nothing if *skip != 0
};
// grid: (nparts, nblk*nblk, count); 256 threads as 16x16; each thread a 4x4 block of a 64x64 tile.
__global__ void __launch_bounds__(256) k_gram(GramArgs a) {
    __shared__ float sa[32][65];
    __shared__ float sb[32][65];
    const int nblk = (a.c + 63) / 64;
    const int bi = blockIdx.y / nblk, bj = blockIdx.y % nblk;
    if (a.skip && *a.skip) return;
    if (!a.X2 && bi > bj) return;  // symmetric: only the upper block triangle
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const float* Xb = a.X + (size_t)blockIdx.z * a.rows * a.c;
    const float* X2b = (a.X2 ? a.X2 : a.X) + (size_t)blockIdx.z * a.rows * a.c;
    const int rbeg = blockIdx.x * GR_ROWS, rend = min(a.rows, rbeg + GR_ROWS);
    if (a.c <= 16) {
        // up to 16 columns (every orthogonalisation of an SSP step): one entry of the c x c block per thread instead of a
        // 4 x 4 patch of a 64 x 64 tile of which 15/16 would be padding
        double s = 0.0;
        for (int r0 = rbeg; r0 < rend; r0 += 32) {
            __syncthreads();
            for (int e = threadIdx.x; e < 32 * 16; e += 256) {
                const int rr = e >> 4, cc = e & 15, grow = r0 + rr;
                const bool in = grow < rend && cc < a.c;
                sa[rr][cc] = in ? Xb[(size_t)grow * a.c + cc] : 0.f;
                sb[rr][cc] = in ? X2b[(size_t)grow * a.c + cc] : 0.f;
            }
            __syncthreads();
#pragma unroll 8
            for (int rr = 0; rr < 32; ++rr) s = fma((double)sa[rr][ty], (double)sb[rr][tx], s);
        }
        if (ty < a.c && tx < a.c) a.part[((size_t)blockIdx.z * a.nparts + blockIdx.x) * a.c * a.c + (size_t)ty * a.c + tx] = s;
        return;
    }
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0;
    for (int r0 = rbeg; r0 < rend; r0 += 32) {
        __syncthreads();
        for (int e = threadIdx.x; e < 32 * 64; e += 256) {
            int rr = e / 64, cc = e % 64;
            int grow = r0 + rr;
            int ca = bi * 64 + cc, cb = bj * 64 + cc;
            sa[rr][cc] = (grow < rend && ca < a.c) ? Xb[(size_t)grow * a.c + ca] : 0.f;
            sb[rr][cc] = (grow < rend && cb < a.c) ? X2b[(size_t)grow * a.c + cb] : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int rr = 0; rr < 32; ++rr) {
            double va[4], vb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                va[i] = (double)sa[rr][ty + 16 * i];
                vb[i] = (double)sb[rr][tx + 16 * i];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fma(va[i], vb[j], acc[i][j]);
        }
    }
    double* out = a.part + ((size_t)blockIdx.z * a.nparts + blockIdx.x) * a.c * a.c;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int ga = bi * 64 + ty + 16 * i, gb = bj * 64 + tx + 16 * j;
            if (ga < a.c && gb < a.c) out[(size_t)ga * a.c + gb] = acc[i][j];
        }
}

// part[c][0][e] <- sum_p part[c][p][e]  (fixed order), so that the single-CTA kernels below read one
// matrix instead of streaming every partial through one SM.  A CTA of 8 warps takes 32 consecutive entries: warp w adds the
// partials p = w (mod 8) of its entries in four independent running sums (256-byte rows, coalesced), the eight warp sums are
// added in a fixed order.  grid: ceil(cc * count / 32), 256 threads.
__global__ void __launch_bounds__(256) k_gram_sum(double* part, int cc, int nparts, int count, const int* skip = nullptr) {
    __shared__ double red[8][33];
    if (skip && *skip) return;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const size_t idx = (size_t)blockIdx.x * 32 + lane;
    const bool in = idx < (size_t)cc * count;
    const size_t c = in ? idx / cc : 0, e = in ? idx % cc : 0;
    double* pb = part + c * (size_t)nparts * cc;
    double s0 = 0.0, s1 = 0.0, s2 = 0.0, s3 = 0.0;
    if (in) {
        int p = w;
        for (; p + 24 < nparts; p += 32) {
            s0 += pb[(size_t)p * cc + e];
            s1 += pb[(size_t)(p + 8) * cc + e];
            s2 += pb[(size_t)(p + 16) * cc + e];
            s3 += pb[(size_t)(p + 24) * cc + e];
        }
        for (; p < nparts; p += 8) s0 += pb[(size_t)p * cc + e];
    }
    red[w][lane] = (s0 + s1) + (s2 + s3);
    __syncthreads();       // every read of partial 0 (warp 0's own) is done before it is overwritten
    if (w == 0 && in) {
        double t = red[0][lane];
#pragma unroll
        for (int k = 1; k < 8; ++k) t += red[k][lane];
        pb[e] = t;
    }
}

// Sum the Gram partials, scale to unit diagonal, Cholesky, invert, and write
// T = D^-1 L^-T (upper triangular, double) so that P~ = P T.  One CTA per matrix.
// Dynamic shared memory: c * chol_ld(c) doubles (rows padded to an odd number of doubles so that
// walking down a column is free of bank conflicts).  NT threads: 256 for the narrow factors of a step; the wide blocks of a
// refresh take chol_threads(c) (every phase is a chain of short dependent steps between barriers, so more warps per
// scheduler shorten it; each entry sees the same operations in the same order whatever NT).
constexpr double CHOL_PIVOT_TOL = 1e-11;  // squared sine of the angle to the previous columns
constexpr int CHOL_NB = 8;                // columns per panel of the factorisation
constexpr int CHOL_IB = 32;               // block size of the triangular inverse
__host__ __device__ inline int chol_ld(int c) { return c | 1; }
__host__ __device__ inline int chol_threads(int c) { return c >= 96 ? 1024 : (c >= 48 ? 512 : 256); }
// `gate` (optional): set to 1 when a scaled pivot^2 falls below gate_tol, i.e. when the columns
// are too ill-conditioned for results derived from W = M^T P to keep float32 accuracy.
// `defic` (optional, [count][c]): 1 for every column whose pivot was rejected (zero or dependent column);
// k_complete replaces those columns of P~ by an orthonormal completion.
template <int NT>
__global__ void __launch_bounds__(NT) k_chol_t(const double* part, double* T, int c, int nparts, int* flags,
                                               int* gate = nullptr, double gate_tol = 0.0, int* defic = nullptr,
                                               const int* skip = nullptr) {
    constexpr int NW = NT / 32;                       // warps; NT / 8 rows per pass inside a panel
    extern __shared__ __align__(16) double Gs[];  // [c][ld]
    if (skip && *skip) return;
    __shared__ double dinv[192], rdiag[192];   // column scaling; reciprocals of the diagonal of L
    __shared__ int dcol[192];
    __shared__ int bad, illc;
    const int tid = threadIdx.x;
    const int ld = chol_ld(c);
    // nparts < 0: the partials were already folded into partial 0 (k_gram_sum); matrices stay |nparts| partials apart
    const int pstride = nparts < 0 ? -nparts : nparts;
    if (nparts < 0) nparts = 1;
    const double* pb = part + (size_t)blockIdx.x * pstride * c * c;
    if (tid == 0) { bad = 0; illc = 0; }
    const int tx = tid & 31, ty = tid >> 5;          // lanes along a row, one row per warp at a time
    for (int i = ty; i < c; i += NW)
        for (int j = tx; j < c; j += 32) {
            int ii = i, jj = j;
            if ((i >> 6) > (j >> 6)) { ii = j; jj = i; }   // lower block triangle was not computed: mirror
            double s = 0.0;
            for (int p = 0; p < nparts; ++p) s += pb[(size_t)p * c * c + (size_t)ii * c + jj];
            Gs[i * ld + j] = s;
        }
    __syncthreads();
    for (int k = tid; k < c; k += NT) {
        double d = Gs[k * ld + k];
        dcol[k] = 0;
        if (!(d > 0.0)) { dinv[k] = 0.0; bad = 1; dcol[k] = 1; } else dinv[k] = 1.0 / sqrt(d);
    }
    __syncthreads();
    for (int i = ty; i < c; i += NW)
        for (int j = tx; j < c; j += 32) {
            double v = Gs[i * ld + j] * dinv[i] * dinv[j];
            if (i == j && dinv[i] == 0.0) v = 1.0;  // zero column: decouple it (fixed up later)
            Gs[i * ld + j] = v;
        }
    __syncthreads();
    // Right-looking Cholesky on the lower triangle, Gs = L L^T, in panels of CHOL_NB columns: a column's update is applied at
    // once only to the rest of its panel (a few entries per thread between barriers); the matrix behind the panel receives the
    // panel's CHOL_NB rank-one updates in one pass (same terms in the same order, one load and store per entry instead of
    // CHOL_NB).  Every thread evaluates the pivot of a column itself (no serial step by one thread, two barriers per column).
    for (int k0 = 0; k0 < c; k0 += CHOL_NB) {
        const int kend = min(c, k0 + CHOL_NB);
        for (int k = k0; k < kend; ++k) {
            double p = Gs[k * ld + k];
            const bool reject = !(p > CHOL_PIVOT_TOL);
            if (tid == 0) {
                if (!(p > gate_tol)) illc = 1;
                if (reject) { bad = 1; dcol[k] = 1; }
            }
            if (reject) p = 1.0;
            const double rl = rsqrt(p);            // 1 / l_kk: all that the later phases need of the diagonal (Gs[k][k] keeps the pivot)
            if (tid == 0) rdiag[k] = rl;
            for (int i = k + 1 + tid; i < c; i += NT) Gs[i * ld + k] = reject ? 0.0 : Gs[i * ld + k] * rl;
            __syncthreads();
            const int w = kend - k - 1;            // columns of the panel still to come
            if (w > 0) {                           // eight threads per row (one per panel column, CHOL_NB = 8), NT / 8 rows per pass
                const int j = k + 1 + (tid & 7);
                if ((tid & 7) < w) {
                    const double ljk = Gs[j * ld + k];
                    for (int i = k + 1 + (tid >> 3); i < c; i += NT / 8)
                        if (i >= j) Gs[i * ld + j] = fma(-Gs[i * ld + k], ljk, Gs[i * ld + j]);
                }
                __syncthreads();
            }
        }
        // behind the panel, one row per warp pass: lanes walk along the row
        if (kend < c) {
            for (int i = kend + (tid >> 5); i < c; i += NW) {
                double li[CHOL_NB];
#pragma unroll
                for (int q = 0; q < CHOL_NB; ++q) li[q] = Gs[i * ld + k0 + q];
                for (int j = kend + (tid & 31); j <= i; j += 32) {
                    double g = Gs[i * ld + j];
#pragma unroll
                    for (int q = 0; q < CHOL_NB; ++q) g = fma(-li[q], Gs[j * ld + k0 + q], g);
                    Gs[i * ld + j] = g;
                }
            }
            __syncthreads();
        }
    }
    // Inverse X = L^-1 of the lower-triangular factor, in blocks of CHOL_IB rows and columns; X[i][j] (i > j) is kept at
    // Gs[j][i] in the unused upper triangle, the diagonal in rdiag.
    // (1) Diagonal blocks, all at once: column j of a block by forward substitution inside the block,
    //     x_j = 1 / l_jj, x_i = -(sum_{k = j}^{i - 1} l_ik x_k) / l_ii; two adjacent lanes share a column and take alternate terms.
    for (int j0 = 0; j0 < c; j0 += NT / 2) {
        const int j = j0 + (tid >> 1), hlf = tid & 1;
        if (j < c) {
            const unsigned pair = 3u << ((tid & 31) & ~1);
            double* xr = Gs + (size_t)j * ld;       // xr[i] = X[i][j] for i > j
            const double xj = rdiag[j];
            const int iend = min(c, (j / CHOL_IB + 1) * CHOL_IB);
            for (int i = j + 1; i < iend; ++i) {
                const double* li = Gs + (size_t)i * ld;
                double s0 = hlf ? 0.0 : li[j] * xj, s1 = 0.0;
                int k = j + 1 + hlf;
                for (; k + 2 < i; k += 4) { s0 = fma(li[k], xr[k], s0); s1 = fma(li[k + 2], xr[k + 2], s1); }
                if (k < i) s0 = fma(li[k], xr[k], s0);
                double sum = s0 + s1;
                sum += __shfl_xor_sync(pair, sum, 1);
                if (!hlf) xr[i] = -sum * rdiag[i];
                __syncwarp(pair);
            }
        }
    }
    __syncthreads();
    // (2) Block rows below the first, one after the other: for the rows a of block row bi and every column b to its left,
    //     S[a][b] = sum_{k = b}^{bi CHOL_IB - 1} l_ak x_kb (parked where X[a][b] will live), then X[a][b] = -sum_{t <= a} x_at S[t][b]
    //     with t running over the rows of the block: two passes in which every entry is independent of the others.
    for (int a0 = CHOL_IB; a0 < c; a0 += CHOL_IB) {
        const int na = min(CHOL_IB, c - a0), ne = na * a0;          // entries (a, b): a0 <= a < a0 + na, b < a0
        for (int e = tid; e < ne; e += NT) {
            const int aa = a0 + e % na, bb = e / na;
            const double* la = Gs + (size_t)aa * ld;
            const double* xb = Gs + (size_t)bb * ld;
            double s0 = la[bb] * rdiag[bb], s1 = 0.0;
            int k = bb + 1;
            for (; k + 1 < a0; k += 2) { s0 = fma(la[k], xb[k], s0); s1 = fma(la[k + 1], xb[k + 1], s1); }
            if (k < a0) s0 = fma(la[k], xb[k], s0);
            Gs[(size_t)bb * ld + aa] = s0 + s1;                     // S[a][b]; nobody reads X[a][b] in this pass
        }
        __syncthreads();
        double xv[(CHOL_IB * 160 + NT - 1) / NT];                   // at most 32 x 160 entries over NT threads
        int q = 0;
        for (int e = tid; e < ne; e += NT, ++q) {
            const int aa = a0 + e % na, bb = e / na;
            const double* sb = Gs + (size_t)bb * ld;                // S[t][b] at sb[t]
            double s0 = rdiag[aa] * sb[aa], s1 = 0.0;               // t = a: x_aa = 1 / l_aa
            int t = a0;
            for (; t + 1 < aa; t += 2) { s0 = fma(Gs[(size_t)t * ld + aa], sb[t], s0); s1 = fma(Gs[(size_t)(t + 1) * ld + aa], sb[t + 1], s1); }
            if (t < aa) s0 = fma(Gs[(size_t)t * ld + aa], sb[t], s0);
            xv[q] = -(s0 + s1);
        }
        __syncthreads();
        q = 0;
        for (int e = tid; e < ne; e += NT, ++q) Gs[(size_t)(e / na) * ld + a0 + e % na] = xv[q];
        __syncthreads();
    }
    // T[j][k] = dinv[j] * Linv[k][j]  for j <= k
    double* Tb = T + (size_t)blockIdx.x * c * c;
    for (int j = ty; j < c; j += NW)
        for (int k = tx; k < c; k += 32)
            Tb[(size_t)j * c + k] = (j < k) ? dinv[j] * Gs[j * ld + k] : (j == k ? dinv[j] * rdiag[j] : 0.0);
    if (defic)
        for (int k = tid; k < c; k += NT) defic[(size_t)blockIdx.x * c + k] = dcol[k];
    if (tid == 0 && bad) atomicOr(flags, 1);
    if (tid == 0 && illc && gate) atomicOr(gate, 1);
}

// Orthonormal completion of a rank-deficient factor (the paper is silent on QR of a rank-deficient P; any
// orthonormal P~ whose span contains range(P) is a valid result).  Every column that k_chol_t rejected is
// replaced by a seeded pseudo-random vector, orthogonalised twice (modified Gram-Schmidt, double sums)
// against the valid columns and normalised.  One CTA per matrix; does nothing unless the status word
// carries PSGD_W_RANK_DEFICIENT.  Ppad (optional) is the padded copy [count][rows][RP] kept in step.
__global__ void __launch_bounds__(256) k_complete(float* Phat, float* Ppad, const int* defic, const int* flags, int rows, int r,
                                                  int RP, uint64_t seed) {
    if (!(*flags & 1)) return;
    __shared__ double red[8];
    __shared__ double bc;
    const int c = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float* Pb = Phat + (size_t)c * rows * r;
    const int* db = defic + (size_t)c * r;
    auto block_sum = [&](double v) -> double {
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();
        if (lane == 0) red[warp] = v;
        __syncthreads();
        if (tid == 0) { double t = 0.0; for (int w = 0; w < 8; ++w) t += red[w]; bc = t; }
        __syncthreads();
        return bc;
    };
    for (int k = 0; k < r; ++k) {
        if (!db[k]) continue;
        for (int row = tid; row < rows; row += 256) {
            uint64_t h = splitmix64(splitmix64(seed ^ (0xC0FFEEull + (uint64_t)c * 1315423911ull + (uint64_t)k)) + (uint64_t)row);
            float u1 = ((float)(uint32_t)(h >> 40) + 0.5f) * (1.0f / 16777216.0f);
            float u2 = ((float)(uint32_t)((h >> 8) & 0xFFFFFF) + 0.5f) * (1.0f / 16777216.0f);
            Pb[(size_t)row * r + k] = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
        }
        __syncthreads();
        for (int pass = 0; pass < 2; ++pass)
            for (int j = 0; j < r; ++j) {
                if (j == k || (db[j] && j > k)) continue;      // columns not yet completed hold nothing useful
                double s = 0.0;
                for (int row = tid; row < rows; row += 256) s += (double)Pb[(size_t)row * r + j] * (double)Pb[(size_t)row * r + k];
                const double cj = block_sum(s);
                for (int row = tid; row < rows; row += 256) Pb[(size_t)row * r + k] -= (float)(cj * (double)Pb[(size_t)row * r + j]);
                __syncthreads();
            }
        double s = 0.0;
        for (int row = tid; row < rows; row += 256) { double v = Pb[(size_t)row * r + k]; s += v * v; }
        const double inv = 1.0 / sqrt(fmax(block_sum(s), 1e-300));
        for (int row = tid; row < rows; row += 256) {
            float v = (float)((double)Pb[(size_t)row * r + k] * inv);
            Pb[(size_t)row * r + k] = v;
            if (Ppad) Ppad[((size_t)c * rows + row) * RP + k] = v;
        }
        __syncthreads();
    }
}

// Xout[row][k] = sum_j X[row][j] * T[j][k]  (double accumulate), k < kout.
// grid: (row tiles of 32, count); 256 threads.  X and Xout may alias (rows are staged).
// (1024 threads per tile, one pass over the items instead of four, were measured on blocks of 128 columns: 113 us against 79 us.)
struct ApplyArgs {
    const float* X;   // [count][rows][c]
    const double* T;  // [count][c][ldt]
    float* Xout;      // [count][rows][kout]
    int rows, c, kout, ldt, upper;
    float* XoutT;     // optional transposed copy [count][kout][rows]
    const int* skip;  // when non-null the kernel does nothing if *skip != 0
};
__global__ void __launch_bounds__(256) k_apply(ApplyArgs a) {
    extern __shared__ __align__(16) float xs[];  // [32][c]
    if (a.skip && *a.skip) return;
    const int row0 = blockIdx.x * 32;
    const float* Xb = a.X + (size_t)blockIdx.y * a.rows * a.c;
    const double* Tb = a.T + (size_t)blockIdx.y * a.c * a.ldt;
    float* Ob = a.Xout + (size_t)blockIdx.y * a.rows * a.kout;
    for (int e = threadIdx.x; e < 32 * a.c; e += 256) {
        int rr = e / a.c, j = e % a.c;
        xs[e] = (row0 + rr < a.rows) ? Xb[(size_t)(row0 + rr) * a.c + j] : 0.f;
    }
    __syncthreads();
    // a thread carries column k of four rows (rr, rr + 8, rr + 16, rr + 24): one load of T[j][k] feeds four independent sums
    for (int e = threadIdx.x; e < 8 * a.kout; e += 256) {
        const int rr = e / a.kout, k = e % a.kout;
        const int jend = a.upper ? min(a.c, k + 1) : a.c;
        double s[4] = {0.0, 0.0, 0.0, 0.0};
        const float* x0 = xs + rr * a.c;
        for (int j = 0; j < jend; ++j) {
            const double t = __ldg(Tb + (size_t)j * a.ldt + k);
#pragma unroll
            for (int q = 0; q < 4; ++q) s[q] = fma((double)x0[q * 8 * a.c + j], t, s[q]);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int row = row0 + rr + 8 * q;
            if (row < a.rows) {
                Ob[(size_t)row * a.kout + k] = (float)s[q];
                if (a.XoutT) a.XoutT[((size_t)blockIdx.y * a.kout + k) * a.rows + row] = (float)s[q];
            }
        }
    }
}

// ----------------------------------------------------------------------------
// Refresh: Rayleigh-Ritz on the block.  A = Z^T Z (double, c x c, summed from Gram
// partials) is diagonalised by cyclic Jacobi with a round-robin pair schedule;
// the r eigenvectors of the largest eigenvalues are written as U [c][r] (double).
// One CTA per matrix; dynamic shared memory: c2*c2 doubles (c2 = c rounded up to even).
// The sweep count is bounded; exhaustion sets PSGD_W_NOT_CONVERGED.
// ----------------------------------------------------------------------------
constexpr int JAC_THREADS = 512;
constexpr int JAC_MAX_SWEEPS = 40;
// stop once the squared off-diagonal norm is this fraction of the squared diagonal norm (1e-11 relative: four orders below
// what the float32 basis built from the eigenvectors can show; the convergence is quadratic, so the sweep that passes the
// test usually ends far below it)
constexpr double JAC_OFF_TOL = 1e-22;
// leading dimension of the shared-memory matrix: odd number of doubles (no bank conflicts down a column)
__host__ __device__ inline int jac_ld(int c2) { return c2 | 1; }
// The eigenvector matrix is kept in shared memory beside A while both fit; wider blocks log their rotations
// (cos, sin per pair and round: the pairs follow from the round-robin schedule) and k_jacobi_vectors replays them.
__host__ __device__ inline bool jac_v_in_smem(int c2) { return (size_t)c2 * jac_ld(c2) * 8 + (size_t)c2 * c2 * 8 <= 200 * 1024; }
__host__ __device__ inline size_t jac_smem_bytes(int c2) {
    return (size_t)c2 * jac_ld(c2) * 8 + (jac_v_in_smem(c2) ? (size_t)c2 * c2 * 8 : 0);
}
// doubles per matrix of the rotation log: a header of 2 + c2 values (sweeps done, unused, order of the eigenvalues), then
// [sweep][round][pair](cos, sin)
__host__ __device__ inline size_t jac_log_doubles(int c2) {
    return jac_v_in_smem(c2) ? 0 : 2 + (size_t)c2 + (size_t)JAC_MAX_SWEEPS * (c2 - 1) * (c2 / 2) * 2;
}
// pair k of round `round` in the round-robin tournament on c2 players: position 0 fixed, the others rotate
__device__ __forceinline__ void jac_pair(int k, int round, int c2, int& p, int& q) {
    const int a0 = (k == 0) ? 0 : 1 + (k - 1 + round) % (c2 - 1);
    const int b0 = 1 + (c2 - 2 - k + round) % (c2 - 1);
    p = min(a0, b0); q = max(a0, b0);
}
__global__ void __launch_bounds__(JAC_THREADS) k_jacobi_top(const double* part, int nparts, int c, int r,
                                                            double* rotlog, double* U, int* flags, const int* skip = nullptr) {
    extern __shared__ __align__(16) double As[];  // [c2][ld] (+ [c2][c2] eigenvectors, transposed, when they fit)
    if (skip && *skip) return;
    __shared__ double cs[128], sn[128];
    __shared__ int pp[128], qq[128];
    __shared__ double offn, diagn;
    __shared__ int order[192];
    const int tid = threadIdx.x;
    const int c2 = (c + 1) & ~1;
    const int ld = jac_ld(c2);
    const int np = c2 / 2;
    const bool vsm = jac_v_in_smem(c2);
    double* Vt = As + (size_t)c2 * ld;                 // Vt[p][i] = V[i][p] (only when vsm)
    double* logb = vsm ? nullptr : rotlog + (size_t)blockIdx.x * jac_log_doubles(c2);
    double* rots = vsm ? nullptr : logb + 2 + c2;
    const int pstride = nparts < 0 ? -nparts : nparts;   // nparts < 0: partials already folded into partial 0
    if (nparts < 0) nparts = 1;
    const double* pb = part + (size_t)blockIdx.x * pstride * c * c;
    for (int e = tid; e < c2 * c2; e += JAC_THREADS) {
        int i = e / c2, j = e % c2;
        double s = 0.0;
        if (i < c && j < c) {
            int ii = i, jj = j;
            if (i / 64 > j / 64) { ii = j; jj = i; }
            for (int p = 0; p < nparts; ++p) s += pb[(size_t)p * c * c + (size_t)ii * c + jj];
        }
        As[i * ld + j] = s;
        if (vsm) Vt[e] = (i == j) ? 1.0 : 0.0;
    }
    __syncthreads();
    // symmetrise (the two triangles of a diagonal block were accumulated separately)
    for (int e = tid; e < c2 * c2; e += JAC_THREADS) {
        int i = e / c2, j = e % c2;
        if (i < j) { double v = 0.5 * (As[i * ld + j] + As[j * ld + i]); As[i * ld + j] = v; As[j * ld + i] = v; }
    }
    __syncthreads();
    int converged = 0, sweeps = 0;
    const int k_first = tid / c2, i_first = tid % c2, k_step = JAC_THREADS / c2, i_step = JAC_THREADS % c2;
    const int ka_first = tid / np, kb_first = tid % np, ka_step = JAC_THREADS / np, kb_step = JAC_THREADS % np;
    for (int sweep = 0; sweep < JAC_MAX_SWEEPS && !converged; ++sweep) {
        for (int round = 0; round < c2 - 1; ++round) {
            if (tid < np) {
                int p, q;
                jac_pair(tid, round, c2, p, q);
                pp[tid] = p; qq[tid] = q;
                double apq = As[p * ld + q], app = As[p * ld + p], aqq = As[q * ld + q];
                double cc = 1.0, ss = 0.0;
                if (fabs(apq) > 1e-300 && fabs(apq) > 1e-18 * sqrt(fabs(app * aqq))) {
                    double tau = (aqq - app) / (2.0 * apq);
                    double t = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
                    cc = 1.0 / sqrt(1.0 + t * t);
                    ss = t * cc;
                }
                cs[tid] = cc; sn[tid] = ss;
                if (!vsm) {
                    double* o = rots + (((size_t)sweep * (c2 - 1) + round) * np + tid) * 2;
                    o[0] = cc; o[1] = ss;
                }
            }
            __syncthreads();
            // A <- J^T A J in one pass over 2 x 2 blocks: the block of pairs (a, b), rows {p_a, q_a} x columns {p_b, q_b}, only
            // needs its own four entries and the two rotations ((a, b) advance without a division)
            for (int e = tid, ka = ka_first, kb = kb_first; e < np * np; e += JAC_THREADS) {
                const int pa = pp[ka], qa = qq[ka], pb2 = pp[kb], qb = qq[kb];
                const double ca = cs[ka], sa = sn[ka], cb = cs[kb], sb = sn[kb];
                const double a00 = As[pa * ld + pb2], a01 = As[pa * ld + qb], a10 = As[qa * ld + pb2], a11 = As[qa * ld + qb];
                // columns: (x_p, x_q) <- (c x_p - s x_q, s x_p + c x_q) with the rotation of pair b
                const double b00 = cb * a00 - sb * a01, b01 = sb * a00 + cb * a01;
                const double b10 = cb * a10 - sb * a11, b11 = sb * a10 + cb * a11;
                // rows: the same with the rotation of pair a
                As[pa * ld + pb2] = ca * b00 - sa * b10;
                As[pa * ld + qb] = ca * b01 - sa * b11;
                As[qa * ld + pb2] = sa * b00 + ca * b10;
                As[qa * ld + qb] = sa * b01 + ca * b11;
                ka += ka_step; kb += kb_step;
                if (kb >= np) { kb -= np; ++ka; }
            }
            if (vsm) {      // V <- V J (thread index runs down the column)
                for (int e = tid, k = k_first, i = i_first; e < np * c2; e += JAC_THREADS) {
                    const int p = pp[k], q = qq[k];
                    const double cc = cs[k], ss = sn[k];
                    const double vip = Vt[p * c2 + i], viq = Vt[q * c2 + i];
                    Vt[p * c2 + i] = cc * vip - ss * viq;
                    Vt[q * c2 + i] = ss * vip + cc * viq;
                    k += k_step; i += i_step;
                    if (i >= c2) { i -= c2; ++k; }
                }
            }
            __syncthreads();
        }
        ++sweeps;
        if (tid == 0) { offn = 0.0; diagn = 0.0; }
        __syncthreads();
        double lo = 0.0, ldg = 0.0;
        for (int e = tid; e < c2 * c2; e += JAC_THREADS) {
            int i = e / c2, j = e % c2;
            double v = As[i * ld + j];
            if (i == j) ldg += v * v; else lo += v * v;
        }
        for (int o = 16; o > 0; o >>= 1) {
            lo += __shfl_xor_sync(0xffffffffu, lo, o);
            ldg += __shfl_xor_sync(0xffffffffu, ldg, o);
        }
        if ((tid & 31) == 0) { atomicAdd(&offn, lo); atomicAdd(&diagn, ldg); }
        __syncthreads();
        converged = (offn <= JAC_OFF_TOL * diagn) || (diagn == 0.0);
        __syncthreads();
    }
    if (tid == 0 && !converged) atomicOr(flags, 2);
    // rank the eigenvalues (descending; ties by index) and emit the top r eigenvectors
    for (int i = tid; i < c2; i += JAC_THREADS) {
        double li = (i < c) ? As[i * ld + i] : -1e300;
        int rank = 0;
        for (int j = 0; j < c2; ++j) {
            double lj = (j < c) ? As[j * ld + j] : -1e300;
            if (lj > li || (lj == li && j < i)) ++rank;
        }
        order[rank] = i;
    }
    __syncthreads();
    if (vsm) {
        double* Ub = U + (size_t)blockIdx.x * c * r;
        for (int e = tid; e < c * r; e += JAC_THREADS) {
            int i = e / r, k = e % r;
            Ub[e] = Vt[order[k] * c2 + i];
        }
    } else {
        if (tid == 0) logb[0] = (double)sweeps;
        for (int i = tid; i < c2; i += JAC_THREADS) logb[2 + i] = (double)order[i];
    }
}

// The eigenvectors of a block too wide for k_jacobi_top's shared memory: V = J_1 J_2 ... replayed from the rotation log.
// Row i of V only ever mixes with itself, and the rotations of one round touch disjoint columns: a CTA carries JV_ROWS rows
// in shared memory, eight lanes share a row and split the pairs of a round between them, a warp-level barrier separates
// the rounds.  The players of the round-robin schedule come from a doubled table (no division per rotation).
constexpr int JV_ROWS = 16, JV_THREADS = 128;
__host__ __device__ inline size_t jacv_smem_bytes(int c2) {
    return (size_t)JV_ROWS * (c2 + 1) * 8 + (size_t)2 * (c2 / 2) * 16 + (size_t)2 * (c2 - 1) * 4;
}
__global__ void __launch_bounds__(JV_THREADS) k_jacobi_vectors(const double* rotlog, int c, int r, double* U, const int* skip = nullptr) {
    extern __shared__ __align__(16) double Vs[];   // [JV_ROWS][c2 + 1], two rounds of (cos, sin), then the table of players
    if (skip && *skip) return;
    const int c2 = (c + 1) & ~1, np = c2 / 2, ldv = c2 + 1;
    double2* rbuf = reinterpret_cast<double2*>(Vs + (size_t)((JV_ROWS * ldv + 1) & ~1));     // [2][np]
    int* perm = reinterpret_cast<int*>(rbuf + 2 * np);                    // perm[j] = 1 + j mod (c2 - 1), j < 2 (c2 - 1)
    const double* logb = rotlog + (size_t)blockIdx.y * jac_log_doubles(c2);
    const double2* rots = reinterpret_cast<const double2*>(logb + 2 + c2);
    const int tid = threadIdx.x, rl = tid >> 3, l8 = tid & 7;
    const int i = blockIdx.x * JV_ROWS + rl;
    for (int j = tid; j < 2 * (c2 - 1); j += JV_THREADS) perm[j] = 1 + j % (c2 - 1);
    double* row = Vs + (size_t)rl * ldv;
    for (int p = l8; p < c2; p += 8) row[p] = (p == i) ? 1.0 : 0.0;
    const int rounds = (int)logb[0] * (c2 - 1);           // the log is one run of rounds, np rotations each
    for (int k = tid; k < np && rounds > 0; k += JV_THREADS) rbuf[k] = __ldg(rots + k);
    __syncthreads();
    for (int g = 0, round = 0; g < rounds; ++g) {
        const double2* cur = rbuf + (g & 1) * np;
        double2 nxt = make_double2(1.0, 0.0);
        if (tid < np && g + 1 < rounds) nxt = __ldg(rots + (size_t)(g + 1) * np + tid);       // np <= JV_THREADS
        for (int k = l8; k < np; k += 8) {
            const int a0 = (k == 0) ? 0 : perm[k - 1 + round], b0 = perm[c2 - 2 - k + round];
            const int p = min(a0, b0), q = max(a0, b0);
            const double2 csn = cur[k];
            const double vp = row[p], vq = row[q];
            row[p] = csn.x * vp - csn.y * vq;
            row[q] = csn.y * vp + csn.x * vq;
        }
        if (tid < np) rbuf[((g + 1) & 1) * np + tid] = nxt;
        __syncthreads();
        if (++round == c2 - 1) round = 0;
    }
    if (i < c) {
        double* Ub = U + (size_t)blockIdx.y * c * r;
        for (int k = l8; k < r; k += 8) Ub[(size_t)i * r + k] = row[(int)logb[2 + k]];
    }
}

// ----------------------------------------------------------------------------
// Stopping test of the refresh: how far the top-r Ritz basis moved between two checks,
//   d^2 = || Pnew - Pold (Pold^T Pnew) ||_F^2   (no cancellation: Pold is orthonormal to float32 rounding).
// k_subspace_change forms the per-row-block sums of squares (S = Pold^T Pnew comes from k_gram / k_gram_sum,
// [r][r] doubles); k_refresh_decide adds them in a fixed order and sets *done when every matrix of the
// handle has stopped moving (rule below).  grid: (ceil(rows / 64), count), 256 threads, r * r floats of dynamic smem.
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_subspace_change(const float* Pold, const float* Pnew, const double* S, size_t s_stride,
                                                         double* dpart, int rows, int r, const int* skip) {
    extern __shared__ __align__(16) float Ss[];   // [r][r]
    __shared__ double red[8];
    if (skip && *skip) return;
    const int c = blockIdx.y, tid = threadIdx.x;
    const double* Sb = S + (size_t)c * s_stride;
    for (int e = tid; e < r * r; e += 256) Ss[e] = (float)Sb[e];
    __syncthreads();
    const int row0 = blockIdx.x * 64;
    const float* po = Pold + (size_t)c * rows * r;
    const float* pn = Pnew + (size_t)c * rows * r;
    double acc = 0.0;
    for (int e = tid; e < 64 * r; e += 256) {
        const int row = row0 + e / r, k = e % r;
        if (row >= rows) continue;
        float v = pn[(size_t)row * r + k];
        for (int j = 0; j < r; ++j) v = fmaf(-po[(size_t)row * r + j], Ss[j * r + k], v);
        acc += (double)v * (double)v;
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if ((tid & 31) == 0) red[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        dpart[(size_t)c * gridDim.x + blockIdx.x] = t;
    }
}
// Rule per matrix (d = movement since the previous check, dprev the one before, q = d / dprev):
//   q < 1 and d q / (1 - q) <= 1e-5: with geometric convergence the movements still to come add up to that
//   (d <= 1e-5 while halving is the case q = 1/2), or
//   d <= 3e-6 (the float32 floor of two Ritz bases computed a few sweeps apart).
__global__ void k_refresh_decide(const double* dpart, int nb, int count, double* dprev, int have_prev, int* done) {
    if (*done) return;
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int all = 1;
    for (int c = 0; c < count; ++c) {
        double t = 0.0;
        for (int b = 0; b < nb; ++b) t += dpart[(size_t)c * nb + b];
        const double d = sqrt(t);
        bool ok = d <= 3e-6;
        if (!ok && have_prev && d < dprev[c]) {
            const double q = d / dprev[c];
            ok = d * q / (1.0 - q) <= 1e-5;
        }
        if (!ok) all = 0;
        dprev[c] = d;
    }
    if (all) *done = 1;
}

}  // namespace psgd
