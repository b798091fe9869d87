// Single-pass ("deferred residual") step kernel and its small finishing kernels.
//
// One SSP-Comp iteration needs every row of every node before P~ exists, and P~ before the
// residual can be formed, which costs three passes over the N*m*n elements when done
// literally.  This kernel does the whole iteration in ONE pass over HBM (read G, read the
// stored Delta of the previous step, write the new Delta = 12 bytes per element):
//
//   * the residual of the previous step is never stored: E_t = Delta_{t-1} - P~_{t-1} Q_{i,t-1}^T is
//     rebuilt on the fly from the small factors (Algorithm 2, last line, folded into Eq. (7a));
//   * a row block's node-mean P[b] = (1/N) sum_i M_i[b,:] Q only needs that row block, so the
//     contraction W_i += M_i[b,:]^T P[b] can follow while the tile is still in shared memory;
//   * because P~ = P T for an upper-triangular T (Cholesky QR), Q_i = M_i^T P~ = W_i T is obtained
//     afterwards from the small matrices alone (k_finish_q), as is P~ itself (k_finish_p).
//
// A thread-block CLUSTER owns a row block of 16 rows for all N nodes; each CTA of the cluster
// owns a column slice, keeps its slice of the tile in shared memory and exchanges the 16 x r
// partial sums of P through distributed shared memory.  Float sums are formed in a fixed
// order everywhere (deterministic results).
#pragma once
#include <cooperative_groups.h>

#include "psgd_kernels.cuh"

namespace psgd {
namespace cg = cooperative_groups;

constexpr int FU_THREADS = 512;
constexpr int FU_R = 16;      // rows per block
constexpr int FU_CH = 64;     // columns per pipeline stage
constexpr int FU_CHP = 68;    // padded stage row stride (floats)
constexpr int FU_STAGES = 3;

struct FusedArgs {
    const float* G;      // [count][N][m][n]
    float* Mbuf;         // [count][N][m][n]  in: Delta_{t-1} (or e_t if !PENDING); out: Delta_t
    const float* Qpad;   // [count][n][RP]    Q_{t-1}, rows padded to RP
    const float* Ppad;   // [count][m][RP]    P~_{t-1}           (PENDING only)
    const float* Qsub;   // [count][N or 1][n][RP] factor the pending residual subtracts (PENDING only)
    const float* Tprev;  // [count][RP][RP] upper-triangular preconditioner, or nullptr (identity)
    float* Pout;         // [count][m][RP]    P' = P * Tprev (node mean, preconditioned)
    float* Wpart;        // [count][KC][N][n][RP]  partial W_i = M_i^T P'
    double* gram;        // [count][KC][r][r]      partial P'^T P'
    int m, n, r, N, KC, CS, Wc, nblk;
    long long qsub_node_stride;  // n*RP, or 0 when all nodes subtract the same factor
};

template <int RP>
__host__ __device__ inline size_t fused_smem_floats(int N, int Wc) {
    size_t Wt = (size_t)Wc + 4;
    size_t tile = (size_t)N * FU_R * Wt;
    size_t stage = (size_t)2 * FU_R * FU_CHP + (size_t)FU_CH * RP + (size_t)FU_R * RP;  // G, Mprev, Qsub chunk, P~prev rows
    size_t qs = (size_t)((Wc + FU_CH - 1) / FU_CH) * FU_CH * RP;   // padded to whole chunks, zero-filled
    size_t red = (size_t)8 * FU_R * RP;
    size_t small = (size_t)2 * FU_R * RP /*Ppart*/ + (size_t)FU_R * RP /*Praw*/ + (size_t)FU_R * RP /*Pb*/ + (size_t)RP * RP /*T*/;
    return tile + FU_STAGES * stage + qs + red + small;
}

template <int RP, bool PENDING>
__global__ void __launch_bounds__(FU_THREADS, 1) k_fused_step(FusedArgs a) {
    extern __shared__ __align__(16) float smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int CS = a.CS, N = a.N, n = a.n, m = a.m, Wc = a.Wc;
    const int q = (int)(blockIdx.x % CS);
    const int cid = (int)(blockIdx.x / CS);
    const int c = cid / a.KC, slot = cid % a.KC;
    const int Wt = Wc + 4;
    const int nch = (Wc + FU_CH - 1) / FU_CH;
    const int colbase = q * Wc;                       // first global column of this CTA
    const int colend = min(n, colbase + Wc);          // one past its last valid column

    // ---- shared memory carve-up ----
    float* tile = smem;                                       // [N][16][Wt]
    float* stg = tile + (size_t)N * FU_R * Wt;                // stages
    constexpr int STG_G = 0, STG_M = FU_R * FU_CHP, STG_Q = 2 * FU_R * FU_CHP, STG_P = STG_Q + FU_CH * RP;
    constexpr int STG_SZ = STG_P + FU_R * RP;
    float* Qs = stg + FU_STAGES * STG_SZ;                     // [nch*64][RP], zero beyond the slice
    float* red = Qs + (size_t)nch * FU_CH * RP;               // [8][16][RP]
    float* Ppart = red + 8 * FU_R * RP;                       // [2][16][RP]
    float* Praw = Ppart + 2 * FU_R * RP;                      // [16][RP]
    float* Pb = Praw + FU_R * RP;                             // [16][RP]
    float* Tp = Pb + FU_R * RP;                               // [RP][RP]

    const float* Gc = a.G + (size_t)c * N * m * n;
    float* Mc = a.Mbuf + (size_t)c * N * m * n;
    const float* Qc = a.Qpad + (size_t)c * n * RP;
    const float* Ppc = PENDING ? a.Ppad + (size_t)c * m * RP : nullptr;
    const float* Qsc = PENDING ? a.Qsub + (size_t)c * (a.qsub_node_stride ? N : 1) * n * RP : nullptr;

    // resident slice of Q_{t-1} and the preconditioner
    for (int e = tid; e < nch * FU_CH * RP / 4; e += FU_THREADS) {
        int col = (e * 4) / RP;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (col < Wc && colbase + col < colend) v = *reinterpret_cast<const float4*>(Qc + (size_t)(colbase + col) * RP + (e * 4) % RP);
        *reinterpret_cast<float4*>(Qs + e * 4) = v;
    }
    const bool precond = a.Tprev != nullptr;
    for (int e = tid; e < RP * RP; e += FU_THREADS) Tp[e] = precond ? a.Tprev[(size_t)c * RP * RP + e] : 0.f;

    // number of row blocks this cluster owns: slot, slot+KC, ...
    const int nb = (a.nblk > slot) ? (a.nblk - slot + a.KC - 1) / a.KC : 0;
    const int per_block = nch * N;
    const int T = nb * per_block;

    auto issue = [&](int s) {   // cp.async loads of stage s (all threads take part)
        int bl = s / per_block, rem = s % per_block;
        int j = rem / N, i = rem % N;
        int row0 = (slot + bl * a.KC) * FU_R;
        float* sb = stg + (s % FU_STAGES) * STG_SZ;
        int cbase = colbase + j * FU_CH;
        if (tid < 256) {
            int rr = tid >> 4, c4 = (tid & 15) * 4;
            int ok = (row0 + rr < m && cbase + c4 < colend) ? 16 : 0;
            size_t off = ok ? ((size_t)i * m + row0 + rr) * n + cbase + c4 : 0;
            cp_async16(sb + STG_G + rr * FU_CHP + c4, Gc + off, ok);
            if (PENDING) {
                // chunk of the factor that the pending residual subtracts: [64 cols][RP]
                for (int e = tid; e < FU_CH * RP / 4; e += 256) {
                    int col = (e * 4) / RP;
                    int okq = (cbase + col < colend) ? 16 : 0;
                    size_t offq = okq ? (size_t)i * a.qsub_node_stride + (size_t)(cbase + col) * RP + (e * 4) % RP : 0;
                    cp_async16(sb + STG_Q + e * 4, Qsc + offq, okq);
                }
            }
        } else {
            int t2 = tid - 256;
            int rr = t2 >> 4, c4 = (t2 & 15) * 4;
            int ok = (row0 + rr < m && cbase + c4 < colend) ? 16 : 0;
            size_t off = ok ? ((size_t)i * m + row0 + rr) * n + cbase + c4 : 0;
            cp_async16(sb + STG_M + rr * FU_CHP + c4, Mc + off, ok);
            if (PENDING && rem == 0) {
                // rows of P~_{t-1} for this block, once per block
                for (int e = t2; e < FU_R * RP / 4; e += 256) {
                    int rr2 = (e * 4) / RP;
                    int okp = (row0 + rr2 < m) ? 16 : 0;
                    size_t offp = okp ? (size_t)(row0 + rr2) * RP + (e * 4) % RP : 0;
                    cp_async16(sb + STG_P + e * 4, Ppc + offp, okp);
                }
            }
        }
    };

    // phase-A mapping: lane -> (row, half); warp -> 4 columns of the chunk; thread -> 2 columns
    const int arow = lane & 15, ahalf = lane >> 4;
    const int acol = warp * 4 + ahalf * 2;  // column within the chunk
    // phase-B mapping: thread -> (node, 4 columns)
    const int Wc4 = Wc / 4;
    const bool btask = tid < N * Wc4;
    const int bnode = btask ? tid / Wc4 : 0;
    const int bcol = btask ? (tid % Wc4) * 4 : 0;   // column within the slice
    const bool bcol_ok = btask && (colbase + bcol < colend);

    float pacc[RP], pprev[RP];
    float wacc[4][RP];
#pragma unroll
    for (int k = 0; k < RP; ++k) { pacc[k] = 0.f; pprev[k] = 0.f; }
#pragma unroll
    for (int jj = 0; jj < 4; ++jj)
#pragma unroll
        for (int k = 0; k < RP; ++k) wacc[jj][k] = 0.f;
    double gacc = 0.0;  // rank 0 only: one entry of P'^T P' per thread

    for (int s = 0; s < FU_STAGES - 1; ++s) {
        if (s < T) issue(s);
        cp_async_commit();
    }
    __syncthreads();   // Qs, Tp visible

    for (int s = 0; s < T; ++s) {
        cp_async_wait<FU_STAGES - 2>();
        __syncthreads();
        if (s + FU_STAGES - 1 < T) issue(s + FU_STAGES - 1);
        cp_async_commit();

        const int bl = s / per_block, rem = s % per_block;
        const int j = rem / N, i = rem % N;
        const int row0 = (slot + bl * a.KC) * FU_R;
        float* sb = stg + (s % FU_STAGES) * STG_SZ;
        if (PENDING && rem == 0) {
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                float4 v = *reinterpret_cast<const float4*>(sb + STG_P + arow * RP + 4 * k4);
                pprev[4 * k4 + 0] = v.x; pprev[4 * k4 + 1] = v.y; pprev[4 * k4 + 2] = v.z; pprev[4 * k4 + 3] = v.w;
            }
        }
        // ---- phase A: M = G + (Mprev - P~prev Qsub^T);  pacc += M Q ----
        {
            float2 g2 = *reinterpret_cast<const float2*>(sb + STG_G + arow * FU_CHP + acol);
            float2 m2 = *reinterpret_cast<const float2*>(sb + STG_M + arow * FU_CHP + acol);
            float mv[2] = {m2.x, m2.y};
            const float gv[2] = {g2.x, g2.y};
#pragma unroll
            for (int cc = 0; cc < 2; ++cc) {
                if (PENDING) {
                    const float* qp = sb + STG_Q + (acol + cc) * RP;
                    float r0 = 0.f, r1 = 0.f, r2 = 0.f, r3 = 0.f;
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        float4 qv = *reinterpret_cast<const float4*>(qp + 4 * k4);
                        r0 = fmaf(pprev[4 * k4 + 0], qv.x, r0);
                        r1 = fmaf(pprev[4 * k4 + 1], qv.y, r1);
                        r2 = fmaf(pprev[4 * k4 + 2], qv.z, r2);
                        r3 = fmaf(pprev[4 * k4 + 3], qv.w, r3);
                    }
                    mv[cc] = mv[cc] - ((r0 + r1) + (r2 + r3));
                }
                mv[cc] += gv[cc];
                const float* qq = Qs + (size_t)(j * FU_CH + acol + cc) * RP;
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    float4 qv = *reinterpret_cast<const float4*>(qq + 4 * k4);
                    pacc[4 * k4 + 0] = fmaf(mv[cc], qv.x, pacc[4 * k4 + 0]);
                    pacc[4 * k4 + 1] = fmaf(mv[cc], qv.y, pacc[4 * k4 + 1]);
                    pacc[4 * k4 + 2] = fmaf(mv[cc], qv.z, pacc[4 * k4 + 2]);
                    pacc[4 * k4 + 3] = fmaf(mv[cc], qv.w, pacc[4 * k4 + 3]);
                }
            }
            if (j * FU_CH + acol < Wc)
                *reinterpret_cast<float2*>(tile + ((size_t)i * FU_R + arow) * Wt + j * FU_CH + acol) = make_float2(mv[0], mv[1]);
        }
        if (rem != per_block - 1) continue;

        // ---- end of a row block: reduce P over the CTA, the cluster, then phase B ----
        const int par = bl & 1;
#pragma unroll
        for (int k = 0; k < RP; ++k) pacc[k] += __shfl_xor_sync(0xffffffffu, pacc[k], 16);
        if (warp >= 8 && lane < 16) {
#pragma unroll
            for (int k = 0; k < RP; ++k) red[((warp - 8) * FU_R + arow) * RP + k] = pacc[k];
        }
        __syncthreads();
        if (warp < 8 && lane < 16) {
#pragma unroll
            for (int k = 0; k < RP; ++k) pacc[k] += red[(warp * FU_R + arow) * RP + k];
        }
        __syncthreads();
        if (warp < 8 && lane < 16) {
#pragma unroll
            for (int k = 0; k < RP; ++k) red[(warp * FU_R + arow) * RP + k] = pacc[k];
        }
        __syncthreads();
        if (tid < FU_R * RP) {
            float sum = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) sum += red[w * FU_R * RP + tid];
            Ppart[par * FU_R * RP + tid] = sum;
        }
        cluster.sync();
        if (tid < FU_R * RP) {
            float sum = 0.f;
            for (int qq = 0; qq < CS; ++qq) {
                const float* rp = cluster.map_shared_rank(Ppart, qq);
                sum += rp[par * FU_R * RP + tid];
            }
            Praw[tid] = sum / (float)N;
        }
        __syncthreads();
        if (tid < FU_R * RP) {
            int rr = tid / RP, k = tid % RP;
            float v;
            if (precond) {
                v = 0.f;
                for (int jj = 0; jj <= k; ++jj) v = fmaf(Praw[rr * RP + jj], Tp[jj * RP + k], v);
            } else {
                v = Praw[tid];
            }
            Pb[tid] = v;
            if (q == 0 && row0 + rr < m) a.Pout[((size_t)c * m + row0 + rr) * RP + k] = v;
        }
        __syncthreads();
        if (q == 0 && tid < a.r * a.r) {
            int ga = tid / a.r, gb = tid % a.r;
#pragma unroll
            for (int rr = 0; rr < FU_R; ++rr) gacc = fma((double)Pb[rr * RP + ga], (double)Pb[rr * RP + gb], gacc);
        }
        // ---- phase B: W_i += M_i[b,:]^T P'[b];  store M ----
        if (btask) {
            const float* tp = tile + (size_t)bnode * FU_R * Wt + bcol;
            float* gout = Mc + ((size_t)bnode * m + row0) * n + colbase + bcol;
#pragma unroll 4
            for (int rr = 0; rr < FU_R; ++rr) {
                float4 v = *reinterpret_cast<const float4*>(tp + rr * Wt);
                if (bcol_ok && row0 + rr < m) *reinterpret_cast<float4*>(gout + (size_t)rr * n) = v;
                const float* pr = Pb + rr * RP;
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    float4 p4 = *reinterpret_cast<const float4*>(pr + 4 * k4);
                    const float pk[4] = {p4.x, p4.y, p4.z, p4.w};
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        wacc[0][4 * k4 + kk] = fmaf(v.x, pk[kk], wacc[0][4 * k4 + kk]);
                        wacc[1][4 * k4 + kk] = fmaf(v.y, pk[kk], wacc[1][4 * k4 + kk]);
                        wacc[2][4 * k4 + kk] = fmaf(v.z, pk[kk], wacc[2][4 * k4 + kk]);
                        wacc[3][4 * k4 + kk] = fmaf(v.w, pk[kk], wacc[3][4 * k4 + kk]);
                    }
                }
            }
        }
#pragma unroll
        for (int k = 0; k < RP; ++k) pacc[k] = 0.f;
    }
    cp_async_wait<0>();

    // ---- flush this cluster's partial W and Gram ----
    if (bcol_ok) {
        float* wp = a.Wpart + ((((size_t)c * a.KC + slot) * N + bnode) * n + colbase + bcol) * RP;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj)
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4)
                *reinterpret_cast<float4*>(wp + (size_t)jj * RP + 4 * k4) =
                    make_float4(wacc[jj][4 * k4 + 0], wacc[jj][4 * k4 + 1], wacc[jj][4 * k4 + 2], wacc[jj][4 * k4 + 3]);
    }
    if (q == 0 && tid < a.r * a.r) a.gram[((size_t)c * a.KC + slot) * a.r * a.r + tid] = gacc;
    cluster.sync();   // nobody leaves while a peer may still read its shared memory
}

// P~ = P' T' (double accumulate).  Writes the user layout [m][r] and the padded copy [m][RP];
// block 0 of each matrix also advances the preconditioner Tacc <- Tprev * T'.
// grid: (ceil(m/64), count), 256 threads.
struct FinishPArgs {
    const float* Pout;   // [count][m][RP]
    const double* T;     // [count][r][r]
    float* Phat;         // [count][m][r]
    float* Ppad;         // [count][m][RP]
    float* Tacc;         // [count][RP][RP]
    int m, r, RP, tprev_identity;
};
__global__ void __launch_bounds__(256) k_finish_p(FinishPArgs a) {
    __shared__ double Ts[16 * 16];
    __shared__ double Tn[16 * 16];
    const int c = blockIdx.y, r = a.r, RP = a.RP;
    const double* Tb = a.T + (size_t)c * r * r;
    for (int e = threadIdx.x; e < r * r; e += 256) Ts[e] = Tb[e];
    __syncthreads();
    const int row0 = blockIdx.x * 64;
    for (int e = threadIdx.x; e < 64 * RP; e += 256) {
        int rr = e / RP, k = e % RP;
        int row = row0 + rr;
        if (row >= a.m) continue;
        double s = 0.0;
        if (k < r) {
            const float* pr = a.Pout + ((size_t)c * a.m + row) * RP;
            for (int j = 0; j <= k; ++j) s = fma((double)pr[j], Ts[j * r + k], s);
            a.Phat[((size_t)c * a.m + row) * r + k] = (float)s;
        }
        a.Ppad[((size_t)c * a.m + row) * RP + k] = (float)s;
    }
    if (blockIdx.x == 0) {
        float* Ta = a.Tacc + (size_t)c * RP * RP;
        for (int e = threadIdx.x; e < r * r; e += 256) {
            int j = e / r, k = e % r;
            double s = 0.0;
            if (a.tprev_identity) s = Ts[e];
            else for (int l = j; l <= k; ++l) s = fma((double)Ta[j * RP + l], Ts[l * r + k], s);
            Tn[e] = s;
        }
        __syncthreads();
        for (int e = threadIdx.x; e < RP * RP; e += 256) {
            int j = e / RP, k = e % RP;
            Ta[e] = (j < r && k < r) ? (float)Tn[j * r + k] : 0.f;
        }
    }
}

// Q_i = (sum over clusters of W_i) T'   (or, when *gate != 0, the sum of the precise
// back-projection partials), Q = (1/N) sum_i Q_i.  Writes the user layouts and the padded
// copies the next fused step reads.  grid: (ceil(n/16), count), 16*RP threads.
struct FinishQArgs {
    const float* Wpart;  // [count][KC][N][n][RP]
    const float* part;   // [count][N][S][n][r]   precise partials (gate != 0)
    const double* T;     // [count][r][r]
    const int* gate;
    float* Qnode;        // [count][N][n][r]
    float* Qmean;        // [count][n][r]
    float* Qpad;         // [count][n][RP]
    float* Qsub;         // [count][N or 1][n][RP]
    int n, r, RP, N, KC, S, sub_is_mean;
};
__global__ void k_finish_q(FinishQArgs a) {
    __shared__ double Ts[16 * 16];
    __shared__ float Ws[16][17];
    const int c = blockIdx.y, r = a.r, RP = a.RP, n = a.n, N = a.N;
    const int cl = threadIdx.x / RP, k = threadIdx.x % RP;
    const int col = blockIdx.x * 16 + cl;
    const bool precise = a.gate && *a.gate != 0;
    const double* Tb = a.T + (size_t)c * r * r;
    for (int e = threadIdx.x; e < r * r; e += blockDim.x) Ts[e] = Tb[e];
    __syncthreads();
    double mean = 0.0;
    for (int i = 0; i < N; ++i) {
        float qv = 0.f;
        if (precise) {
            if (col < n && k < r) {
                float s = 0.f;
                for (int sl = 0; sl < a.S; ++sl) s += a.part[((((size_t)c * N + i) * a.S + sl) * n + col) * r + k];
                qv = s;
            }
        } else {
            float w = 0.f;
            if (col < n)
                for (int sl = 0; sl < a.KC; ++sl) w += a.Wpart[((((size_t)c * a.KC + sl) * N + i) * n + col) * RP + k];
            __syncthreads();
            Ws[cl][k] = w;
            __syncthreads();
            if (col < n && k < r) {
                double s = 0.0;
                for (int j = 0; j <= k; ++j) s = fma((double)Ws[cl][j], Ts[j * r + k], s);
                qv = (float)s;
            }
        }
        if (col < n) {
            if (k < r) a.Qnode[(((size_t)c * N + i) * n + col) * r + k] = qv;
            if (!a.sub_is_mean) a.Qsub[(((size_t)c * N + i) * n + col) * RP + k] = (k < r) ? qv : 0.f;
        }
        mean += (double)qv;
    }
    if (col < n) {
        float qm = (float)(mean / (double)N);
        if (k < r) a.Qmean[((size_t)c * n + col) * r + k] = qm;
        a.Qpad[((size_t)c * n + col) * RP + k] = (k < r) ? qm : 0.f;
        if (a.sub_is_mean) a.Qsub[((size_t)c * n + col) * RP + k] = (k < r) ? qm : 0.f;
    }
}

// Padded copies of the state for the fused kernel: Qpad [count][n][RP] from Q [count][n][r].
__global__ void k_pad_rows(const float* X, float* Xpad, size_t rows, int r, int RP) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * RP) return;
    size_t row = idx / RP;
    int k = (int)(idx % RP);
    Xpad[idx] = (k < r) ? X[row * r + k] : 0.f;
}

}  // namespace psgd
