// Single-pass ("deferred residual") step kernel and its small finishing kernels.
//
// One SSP-Comp iteration needs every row of every node before P~ exists, and P~ before the
// residual can be formed, which costs three passes over the N*m*n elements when done
// literally.  This kernel does the whole iteration in ONE pass over HBM (read G, read the
// stored Delta of the previous step, write the new Delta = 12 bytes per element):
//
//   * the residual of the previous step is never stored: the buffer holds Delta_{t-1} and
//     e_t = Delta_{t-1} - P~_{t-1} Q_{i,t-1}^T is rebuilt from the small factors (Algorithm 2,
//     last line, folded into Eq. (7a)):  Delta_t = S - P~_{t-1} Qsub_i^T  with  S = g_t + Delta_{t-1};
//   * the projection is linear, so it is taken of S and corrected in the small space:
//         P = (1/N) sum_i Delta_t,i Q = (1/N) sum_i S_i Q  -  P~_{t-1} C,   C = (1/N) sum_i Qsub_i^T Q  (r x r);
//   * a row block's P only needs that row block, so the contraction W_i += Delta_t,i[b,:]^T P[b]
//     follows while the block is still in shared memory;
//   * because P~ = P T for an upper-triangular T (Cholesky QR), Q_i = Delta_i^T P~ = W_i T is obtained
//     afterwards from the small matrices alone (k_finish_q), as is P~ itself (k_finish_p).  The
//     previous step's accumulated T is folded into Q beforehand (Q' = Q T), so that P' = P T
//     comes out nearly orthonormal and W = Delta^T P' keeps float32 accuracy.
//
// A thread-block CLUSTER owns row blocks of 8 rows for all N nodes; each CTA of the cluster
// owns a column slice of WC columns.  G and the stored Delta arrive as TMA tiles (8 rows x up to
// 256 columns of one node, cp.async.bulk.tensor with zero fill beyond the matrix edges) in a
// ring of shared-memory stages whose completion is tracked by mbarriers; the warps take turns
// issuing the copies.  S is kept in a double-buffered shared-memory tile; the 8 x r partial
// sums of P are pushed to the peers' shared memory (DSMEM) and the cluster barrier is split
// into arrive / wait so that its latency is covered by the next block's loads and arithmetic.
// Float sums are formed in a fixed order everywhere (bit-reproducible results).  Every
// mbarrier wait is bounded; a wait that runs out sets PSGD_W_TIMEOUT in the status word and
// the kernel carries on to its end.
#pragma once
#include <cooperative_groups.h>
#include <cuda.h>

#include "psgd_kernels.cuh"

namespace psgd {
namespace cg = cooperative_groups;

constexpr int FU_THREADS = 256;
constexpr int FU_R = 8;        // rows per block
constexpr int FU_RG = 4;       // rows per warp task
constexpr int FU_MAXCS = 8;    // largest cluster
constexpr unsigned FU_WAIT_LIMIT = 1u << 20;   // polls of one mbarrier wait before giving up
constexpr int FU_W_TIMEOUT = 4;                // == PSGD_W_TIMEOUT

struct FusedArgs {
    float* Mbuf;         // [count][N][m][n]  in: Delta_{t-1} (or e_t if !PENDING); out: Delta_t
    const float* Qpad;   // [count][n][RP]    Q' = Q_{t-1} T (preconditioned), rows padded to RP
    const float* Ppad;   // [count][m][RP]    P~_{t-1}           (PENDING only)
    const float* Qsub;   // [count][N or 1][n][RP] factor the pending residual subtracts (PENDING only)
    const float* Cmat;   // [count][RP][RP]   C' = mean_i Qsub_i^T Q'                    (PENDING only)
    float* Pout;         // [count][m][RP]    P' = P T (node mean, preconditioned)
    float* Wpart;        // [count][KC][N][n][RP]  partial W_i = Delta_i^T P'
    double* gram;        // [count][KC][r][r]      partial P'^T P'
    int* flags;          // device status word
    int m, n, r, N, KC, CS, nblk;
    long long qsub_node_stride;  // n*RP, or 0 when all nodes subtract the same factor
};

template <int WC>
struct FusedGeom {
    static constexpr int BW = WC >= 256 ? 256 : WC;      // columns of one TMA tile = one stage
    static constexpr int NH = WC / BW;                   // stages per node and block
    static constexpr int CPL = BW / 128;                 // columns per lane in the projection phase
    static constexpr int NCG = 4;                        // column groups per stage (one warp each, two row groups)
    static constexpr int NST = BW == 256 ? 5 : 8;        // ring depth
    static constexpr int TPN = WC / 8;                   // back-projection threads per node
    static constexpr int STAGE_FLOATS = 2 * FU_R * BW;   // G tile, then stored-Delta tile
};

template <int RP, int WC>
__host__ __device__ inline size_t fused_smem_bytes(int N) {
    using Ge = FusedGeom<WC>;
    size_t fl = (size_t)2 * N * FU_R * WC            // S tile, double-buffered
              + (size_t)Ge::NST * Ge::STAGE_FLOATS   // ring
              + (size_t)2 * 2 * Ge::NH * Ge::NCG * 32   // per-warp partial sums of P
              + (size_t)2 * FU_MAXCS * FU_R * RP     // partial sums received from the cluster
              + (size_t)2 * FU_R * RP                // P' rows
              + (size_t)2 * FU_R * RP                // P~_{t-1} rows
              + (size_t)RP * RP;                     // C'
    return fl * 4 + (size_t)(2 * Ge::NST + 2) * 8 + 128;   // + alignment slack for the TMA destinations
}

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after FU_WAIT_LIMIT polls, records it and lets the caller go on; a thread
// that has given up once no longer waits at all (`dead`), so a broken pipeline still ends quickly.
__device__ __forceinline__ void mbar_wait(unsigned bar, unsigned parity, int* flags, bool& dead) {
    if (dead) return;
    for (unsigned it = 0; it < FU_WAIT_LIMIT; ++it)
        if (mbar_try_wait(bar, parity)) return;
    dead = true;
    atomicOr(flags, FU_W_TIMEOUT);
}
// TMA: one tile {x: columns, y: rows, z: (matrix, node)} of a rank-3 tensor map into shared memory.
// x must be a multiple of 4 floats (16 bytes); coordinates past the extents read zeros.
__device__ __forceinline__ void tma_load_3d(unsigned dst, const CUtensorMap* map, int x, int y, int z, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
__device__ __forceinline__ void cluster_arrive_release() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void cluster_wait_acquire() {
    asm volatile("barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void st_cluster_f32(unsigned local_addr, unsigned rank, float v) {
    unsigned remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;\n" ::"r"(remote), "f"(v) : "memory");
}

// Sum over the 32 lanes of NV per-lane values with a halving butterfly (fixed order).
// On return lane l holds the total of value index l (NV == 32) or l >> 1 (NV == 16) in v[0].
template <int NV>
__device__ __forceinline__ void butterfly_reduce(float (&v)[NV], int lane) {
#pragma unroll
    for (int o = 16, cnt = NV; cnt > 1; o >>= 1, cnt >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int j = 0; j < cnt / 2; ++j) {
            float send = up ? v[j] : v[j + cnt / 2];
            float keep = up ? v[j + cnt / 2] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    if (NV == 16) v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
}

// d = a * b + c on two packed floats (one instruction slot on sm_100)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n.reg .b64 ra, rb, rc, rd;\n"
        "mov.b64 ra, {%2, %3};\nmov.b64 rb, {%4, %5};\nmov.b64 rc, {%6, %7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\n"
        "mov.b64 {%0, %1}, rd;\n}\n"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}

// A float delivered to a peer CTA's shared memory; the peer's mbarrier counts the 4 bytes.
__device__ __forceinline__ void st_async_cluster_f32(unsigned local_addr, unsigned local_bar, unsigned rank, float v) {
    unsigned raddr, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(raddr) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(rbar) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];\n"
                 ::"r"(raddr), "r"(__float_as_uint(v)), "r"(rbar) : "memory");
}

template <int RP, int WC, bool PENDING>
__global__ void __launch_bounds__(FU_THREADS, 1)
k_fused_step(const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmM, FusedArgs a) {
    using Ge = FusedGeom<WC>;
    constexpr int BW = Ge::BW, NH = Ge::NH, CPL = Ge::CPL, NCG = Ge::NCG, NST = Ge::NST, TPN = Ge::TPN;
    constexpr int NV = FU_RG * RP;         // per-lane partial sums of one warp task
    constexpr int PR = FU_R * RP;          // entries of one block of P
    constexpr int RP2 = RP / 2;
    constexpr unsigned STAGE_BYTES = Ge::STAGE_FLOATS * 4;

    extern __shared__ __align__(16) float smem_raw[];
    float* smem = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    cg::cluster_group cluster = cg::this_cluster();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int CS = a.CS, N = a.N, n = a.n, m = a.m;
    const int q = (int)(blockIdx.x % CS);              // rank in the cluster = column slice
    const int cid = (int)(blockIdx.x / CS);
    const int c = cid / a.KC, slot = cid % a.KC;
    const int colbase = q * WC;
    const int colend = min(n, colbase + WC);
    const int ncols = max(0, colend - colbase);

    // ---- shared memory carve-up ----
    float* ring = smem;                                        // [NST][2][8][BW]   (128-byte aligned)
    float* tile = ring + (size_t)NST * Ge::STAGE_FLOATS;       // [2][N][8][WC]
    float* PpartW = tile + (size_t)2 * N * FU_R * WC;          // [2][2][NH*NCG][32]
    float* Precv = PpartW + 2 * 2 * NH * NCG * 32;             // [2][FU_MAXCS][PR]
    float* Pb = Precv + 2 * FU_MAXCS * PR;                     // [2][PR]   P' rows
    float* Pp = Pb + 2 * PR;                                   // [2][PR]   P~_{t-1} rows
    float* Cm = Pp + 2 * PR;                                   // [RP][RP]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(Cm + RP * RP);
    const unsigned bar_full = smem_u32(bars), bar_empty = smem_u32(bars + NST), bar_recv = smem_u32(bars + 2 * NST);

    float* Mc = a.Mbuf + (size_t)c * N * m * n;
    const float* Qc = a.Qpad + (size_t)c * n * RP;
    const float* Ppc = PENDING ? a.Ppad + (size_t)c * m * RP : nullptr;
    const float* Qsc = PENDING ? a.Qsub + (size_t)c * (a.qsub_node_stride ? N : 1) * n * RP : nullptr;

    // row blocks this cluster owns: slot, slot + KC, ...
    const int nb = (a.nblk > slot) ? (a.nblk - slot + a.KC - 1) / a.KC : 0;
    const int nstb = NH * N;               // stages per block: column half outer, node inner
    const int T = nb * nstb;

    // ---- one-time set-up ----
    if (tid == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, FU_THREADS / 32);
        }
        mbar_init(bar_recv, 1);
        mbar_init(bar_recv + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (PENDING)
        for (int e = tid; e < RP * RP; e += FU_THREADS) Cm[e] = a.Cmat[(size_t)c * RP * RP + e];
    cluster.sync();   // every CTA's barriers exist before a peer sends to them
    bool dead = false;

    // projection phase: warp -> (column group, row group) of a stage, lane -> CPL adjacent columns
    const int cgp = warp % NCG, rgl = warp / NCG;
    const int acol = cgp * 32 * CPL + lane * CPL;      // column within the stage
    // back-projection phase: thread -> (node, 4 + 4 columns)
    const int bi = tid / TPN, tc = tid % TPN;
    const bool btask = bi < N;
    const int bc0 = 4 * tc, bc1 = WC / 2 + 4 * tc;
    const bool bok0 = btask && bc0 < ncols, bok1 = btask && bc1 < ncols;
    float2 wacc[8][RP2];                   // W for 8 columns, pairs over k
    constexpr int QSN = PENDING ? 4 : 1;
    float2 qs[QSN][RP];                    // Qsub for column pairs (2j, 2j+1), per k
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
        for (int k = 0; k < RP2; ++k) wacc[j][k] = make_float2(0.f, 0.f);
    if (PENDING) {
        float t8[8][RP];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int col = (j < 4 ? bc0 : bc1) + (j & 3);
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (btask && col < ncols)
                    v = __ldg(reinterpret_cast<const float4*>(Qsc + (size_t)bi * a.qsub_node_stride + (size_t)(colbase + col) * RP + 4 * k4));
                t8[j][4 * k4 + 0] = v.x; t8[j][4 * k4 + 1] = v.y; t8[j][4 * k4 + 2] = v.z; t8[j][4 * k4 + 3] = v.w;
            }
        }
#pragma unroll
        for (int j2 = 0; j2 < QSN; ++j2)
#pragma unroll
            for (int k = 0; k < RP; ++k) qs[j2][k] = make_float2(t8[(2 * j2) % 8][k], t8[(2 * j2 + 1) % 8][k]);
    }

    // ---- producer role (taken in turn by the warps): two TMA tiles per stage ----
    // state of the next stage to issue, advanced by every thread in step with the main loop
    int p_bl = 0, p_h = 0, p_i = 0, p_ss = 0, p_par = 1;   // p_par: parity of the slot's previous release
    auto issue_next = [&]() {      // called by one whole warp; the slot must have been released
        if (lane == 0) {
            const int row = (slot + p_bl * a.KC) * FU_R;
            const unsigned bar = bar_full + 8 * p_ss;
            const unsigned dst = smem_u32(ring + (size_t)p_ss * Ge::STAGE_FLOATS);
            mbar_expect_tx(bar, STAGE_BYTES);
            tma_load_3d(dst, &tmG, colbase + p_h * BW, row, c * N + p_i, bar);
            tma_load_3d(dst + STAGE_BYTES / 2, &tmM, colbase + p_h * BW, row, c * N + p_i, bar);
        }
        __syncwarp();
    };
    auto advance_next = [&]() {
        if (++p_i == N) { p_i = 0; if (++p_h == NH) { p_h = 0; ++p_bl; } }
        if (++p_ss == NST) { p_ss = 0; p_par ^= 1; }
    };
    // The ring runs NST - 2 stages ahead: the slot refilled at stage sg is the one released two stages
    // earlier, so the warp on duty practically never waits for a slower warp.
    for (int s = 0; s < NST - 2; ++s) {
        if (s < T && warp == 0) issue_next();
        advance_next();
    }

    // P' of one finished block: node mean of the received partial sums, small-space correction.
    // Every thread waits for the cluster's partial sums itself (bounded), so no barrier follows the wait.
    auto finish_block = [&](int bl) {
        const int pb = bl & 1;
        const int prow0 = (slot + bl * a.KC) * FU_R;
        mbar_wait(bar_recv + 8 * pb, (unsigned)((bl >> 1) & 1), a.flags, dead);
        if (tid < PR) {
            const int rr = tid / RP, k = tid % RP;
            float sum = 0.f;
            for (int qq = 0; qq < CS; ++qq) sum += Precv[(pb * FU_MAXCS + qq) * PR + tid];
            float v = sum / (float)N;
            if (PENDING) {
                const float* pp = Pp + pb * PR + rr * RP;
#pragma unroll
                for (int j = 0; j < RP; ++j) v = fmaf(-pp[j], Cm[j * RP + k], v);
            }
            if (prow0 + rr >= m) v = 0.f;
            Pb[pb * PR + tid] = v;
            if (q == 0 && prow0 + rr < m) a.Pout[((size_t)c * m + prow0 + rr) * RP + k] = v;
        }
        __syncthreads();
    };
    double gacc = 0.0;   // rank 0, threads 64 .. 64 + r*r: one entry of P'^T P'
    auto gram_block = [&](int bl) {
        const int pb = bl & 1;
        const int t2 = tid - 64;
        if (q == 0 && t2 >= 0 && t2 < a.r * a.r) {
            const int ga = t2 / a.r, gb = t2 % a.r;
#pragma unroll
            for (int rr = 0; rr < FU_R; ++rr)
                gacc = fma((double)Pb[pb * PR + rr * RP + ga], (double)Pb[pb * PR + rr * RP + gb], gacc);
        }
    };
    // back-projection of row rr of block bl: Delta = S - P~_{t-1} Qsub^T, W += Delta^T P', store Delta
    auto back_row = [&](int bl, int rr) {
        if (!btask) return;
        const int pb = bl & 1;
        const int prow = (slot + bl * a.KC) * FU_R + rr;
        const float* tp = tile + (((size_t)pb * N + bi) * FU_R + rr) * WC;
        const float4 v0 = *reinterpret_cast<const float4*>(tp + bc0);
        const float4 v1 = *reinterpret_cast<const float4*>(tp + bc1);
        float2 mv[4] = {make_float2(v0.x, v0.y), make_float2(v0.z, v0.w), make_float2(v1.x, v1.y), make_float2(v1.z, v1.w)};
        if (PENDING) {
            const float* pp = Pp + pb * PR + rr * RP;
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                const float4 p4 = *reinterpret_cast<const float4*>(pp + 4 * k4);
                const float pk[4] = {-p4.x, -p4.y, -p4.z, -p4.w};
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const float2 pd = make_float2(pk[kk], pk[kk]);
#pragma unroll
                    for (int j2 = 0; j2 < 4; ++j2) mv[j2] = ffma2(pd, qs[j2 % QSN][4 * k4 + kk], mv[j2]);
                }
            }
        }
        const float* pr = Pb + pb * PR + rr * RP;
        float2 pk2[RP2];
#pragma unroll
        for (int k4 = 0; k4 < RP / 4; ++k4) {
            const float4 p4 = *reinterpret_cast<const float4*>(pr + 4 * k4);
            pk2[2 * k4] = make_float2(p4.x, p4.y);
            pk2[2 * k4 + 1] = make_float2(p4.z, p4.w);
        }
#pragma unroll
        for (int j2 = 0; j2 < 4; ++j2) {
            const float2 mx = make_float2(mv[j2].x, mv[j2].x), my = make_float2(mv[j2].y, mv[j2].y);
#pragma unroll
            for (int k2 = 0; k2 < RP2; ++k2) {
                wacc[2 * j2][k2] = ffma2(mx, pk2[k2], wacc[2 * j2][k2]);
                wacc[2 * j2 + 1][k2] = ffma2(my, pk2[k2], wacc[2 * j2 + 1][k2]);
            }
        }
        if (prow < m) {
            float* go = Mc + ((size_t)bi * m + prow) * n + colbase;
            if (bok0) *reinterpret_cast<float4*>(go + bc0) = make_float4(mv[0].x, mv[0].y, mv[1].x, mv[1].y);
            if (bok1) *reinterpret_cast<float4*>(go + bc1) = make_float4(mv[2].x, mv[2].y, mv[3].x, mv[3].y);
        }
    };

    float2 sacc[FU_RG][RP2];
#pragma unroll
    for (int rr = 0; rr < FU_RG; ++rr)
#pragma unroll
        for (int k = 0; k < RP2; ++k) sacc[rr][k] = make_float2(0.f, 0.f);
    float2 Qr[CPL][RP2];     // rows of Q' for this lane's columns of the current column half, pairs over k
    float pprev_reg = 0.f;   // thread < PR: its entry of P~_{t-1} for the block being projected

    const int k0 = nstb / 2;            // stage of a block at which the previous block's P' is finished
    const int span = nstb - k0;         // stages over which the previous block's 8 rows are back-projected
    int ss = 0, par = 0;                // ring slot and parity of the stage being consumed
    int sg = 0;
    for (int bl = 0; bl < nb; ++bl) {
        const int row0 = (slot + bl * a.KC) * FU_R;
        const int pbuf = bl & 1;
        int brow = 0, bacc = 0;         // rows of the previous block done so far; Bresenham accumulator
        if (tid == 0) mbar_expect_tx(bar_recv + 8 * pbuf, (unsigned)(CS * PR * 4));
        if (PENDING && tid < PR) {
            const int rr = tid / RP;
            pprev_reg = (row0 + rr < m) ? __ldg(Ppc + (size_t)(row0 + rr) * RP + tid % RP) : 0.f;
        }
        int sl = 0;
        for (int h = 0; h < NH; ++h) {
            if (NH > 1 || bl == 0) {   // (re)load this lane's rows of Q' for the column half
#pragma unroll
                for (int j = 0; j < CPL; ++j)
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const int col = h * BW + acol + j;
                        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (col < ncols) v = __ldg(reinterpret_cast<const float4*>(Qc + (size_t)(colbase + col) * RP + 4 * k4));
                        Qr[j][2 * k4] = make_float2(v.x, v.y);
                        Qr[j][2 * k4 + 1] = make_float2(v.z, v.w);
                    }
            }
            for (int i = 0; i < N; ++i, ++sl, ++sg) {
                if (warp == (sg & 7)) {           // this warp's turn to refill the ring
                    if (sg + NST - 2 < T) {
                        if (sg > 1) mbar_wait(bar_empty + 8 * p_ss, (unsigned)p_par, a.flags, dead);
                        issue_next();
                    }
                }
                advance_next();
                if (bl > 0 && sl == k0) {
                    finish_block(bl - 1);
                    gram_block(bl - 1);
                }

                // ---- projection: S = g + stored Delta -> tile; sacc += S Q' ----
                mbar_wait(bar_full + 8 * ss, (unsigned)par, a.flags, dead);
                {
                    const float* sgp = ring + (size_t)ss * Ge::STAGE_FLOATS + (size_t)(rgl * FU_RG) * BW + acol;
                    const float* smp = sgp + FU_R * BW;
                    float* tp = tile + (((size_t)pbuf * N + i) * FU_R + rgl * FU_RG) * WC + h * BW + acol;
                    float sv[FU_RG][CPL];
#pragma unroll
                    for (int rr = 0; rr < FU_RG; ++rr) {
                        if (CPL == 2) {
                            const float2 g2 = *reinterpret_cast<const float2*>(sgp + rr * BW);
                            const float2 m2 = *reinterpret_cast<const float2*>(smp + rr * BW);
                            sv[rr][0] = g2.x + m2.x; sv[rr][CPL - 1] = g2.y + m2.y;
                        } else {
                            sv[rr][0] = sgp[rr * BW] + smp[rr * BW];
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * ss);   // the stage is in registers: release the slot
#pragma unroll
                    for (int rr = 0; rr < FU_RG; ++rr) {
                        if (CPL == 2) *reinterpret_cast<float2*>(tp + rr * WC) = make_float2(sv[rr][0], sv[rr][CPL - 1]);
                        else tp[rr * WC] = sv[rr][0];
#pragma unroll
                        for (int j = 0; j < CPL; ++j) {
                            const float2 sd = make_float2(sv[rr][j], sv[rr][j]);
#pragma unroll
                            for (int k2 = 0; k2 < RP2; ++k2) sacc[rr][k2] = ffma2(sd, Qr[j][k2], sacc[rr][k2]);
                        }
                    }
                }
                if (++ss == NST) { ss = 0; par ^= 1; }

                if (i == N - 1) {   // the column half is complete for every node: reduce over the warp's columns
                    float v[NV];
#pragma unroll
                    for (int rr = 0; rr < FU_RG; ++rr)
#pragma unroll
                        for (int k2 = 0; k2 < RP2; ++k2) {
                            v[rr * RP + 2 * k2] = sacc[rr][k2].x;
                            v[rr * RP + 2 * k2 + 1] = sacc[rr][k2].y;
                            sacc[rr][k2] = make_float2(0.f, 0.f);
                        }
                    butterfly_reduce<NV>(v, lane);
                    if (NV == 32 || (lane & 1) == 0)
                        PpartW[((pbuf * 2 + rgl) * (NH * NCG) + h * NCG + cgp) * 32 + (NV == 32 ? lane : lane >> 1)] = v[0];
                }

                // ---- back-projection of the previous block, spread over this block's stages ----
                if (bl > 0 && sl >= k0) {
                    bacc += FU_R;
                    while (bacc >= span && brow < FU_R) { back_row(bl - 1, brow); ++brow; bacc -= span; }
                }
            }
        }
        // block projected: CTA sum of the partial P, sent to every CTA of the cluster
        if (PENDING && tid < PR) Pp[pbuf * PR + tid] = pprev_reg;
        __syncthreads();
        if (tid < PR) {
            const int rr = tid / RP, k = tid % RP;
            const int rgi = rr / FU_RG, j = (rr % FU_RG) * RP + k;
            float sum = 0.f;
#pragma unroll
            for (int g = 0; g < NH * NCG; ++g) sum += PpartW[((pbuf * 2 + rgi) * (NH * NCG) + g) * 32 + j];
            const unsigned dst = smem_u32(Precv + (pbuf * FU_MAXCS + q) * PR + tid);
            for (int qq = 0; qq < CS; ++qq) st_async_cluster_f32(dst, bar_recv + 8 * pbuf, (unsigned)qq, sum);
        }
    }
    if (nb > 0) {
        finish_block(nb - 1);
        gram_block(nb - 1);
#pragma unroll 1
        for (int rr = 0; rr < FU_R; ++rr) back_row(nb - 1, rr);
    }

    // ---- flush this cluster's partial W and Gram ----
    if (btask) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int col = (j < 4 ? bc0 : bc1) + (j & 3);
            if (col < ncols) {
                float* wp = a.Wpart + ((((size_t)c * a.KC + slot) * N + bi) * n + colbase + col) * RP;
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4)
                    *reinterpret_cast<float4*>(wp + 4 * k4) =
                        make_float4(wacc[j][2 * k4].x, wacc[j][2 * k4].y, wacc[j][2 * k4 + 1].x, wacc[j][2 * k4 + 1].y);
            }
        }
    }
    {
        const int t2 = tid - 64;
        if (q == 0 && t2 >= 0 && t2 < a.r * a.r) a.gram[((size_t)c * a.KC + slot) * a.r * a.r + t2] = gacc;
    }
    cluster.sync();   // nobody leaves while a peer may still address its shared memory
}

// P~ = P' T' (double accumulate).  Writes the user layout [m][r] and the padded copy [m][RP];
// block 0 of each matrix also advances the accumulated transform Tacc <- Tacc * T'.
// grid: (ceil(m/64), count), 256 threads.
struct FinishPArgs {
    const float* Pout;   // [count][m][RP]
    const double* T;     // [count][r][r]
    float* Phat;         // [count][m][r]
    float* Ppad;         // [count][m][RP]
    const float* Tacc_in;   // [count][RP][RP]  (ignored when tprev_identity)
    float* Tacc_out;        // [count][RP][RP]
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
        const float* Ti = a.Tacc_in + (size_t)c * RP * RP;
        float* To = a.Tacc_out + (size_t)c * RP * RP;
        for (int e = threadIdx.x; e < r * r; e += 256) {
            int j = e / r, k = e % r;
            double s = 0.0;
            if (a.tprev_identity) s = Ts[e];
            else for (int l = j; l <= k; ++l) s = fma((double)Ti[j * RP + l], Ts[l * r + k], s);
            Tn[e] = s;
        }
        __syncthreads();
        for (int e = threadIdx.x; e < RP * RP; e += 256) {
            int j = e / RP, k = e % RP;
            To[e] = (j < r && k < r) ? (float)Tn[j * r + k] : 0.f;
        }
    }
}

// Q_i = (sum over clusters of W_i) T'   (or, when *gate != 0, the sum of the precise
// back-projection partials), Q = (1/N) sum_i Q_i.  Writes the user layouts, the factor the
// pending residual subtracts (Qsub), the preconditioned basis Q' = Q Tacc the next fused step
// projects with, and this block's share of C' = mean_i Qsub_i^T Q'.
// grid: (ceil(n/16), count), 16*RP threads.
struct FinishQArgs {
    const float* Wpart;  // [count][KC][N][n][RP]
    const float* part;   // [count][N][S][n][r]   precise partials (gate != 0)
    const double* T;     // [count][r][r]
    const float* Tacc;   // [count][RP][RP]  accumulated transform (already advanced by k_finish_p)
    const int* gate;
    float* Qnode;        // [count][N][n][r]
    float* Qmean;        // [count][n][r]
    float* Qpad;         // [count][n][RP]   Q'
    float* Qsub;         // [count][N or 1][n][RP]
    double* Cpart;       // [count][nblocks][RP][RP]
    int n, r, RP, N, KC, S, sub_is_mean;
};
__global__ void k_finish_q(FinishQArgs a) {
    __shared__ double Ts[16 * 16];
    __shared__ float Ta[16 * 16];
    __shared__ float Ws[16][17];
    __shared__ float Qs_[16][17];     // Q' of this block's columns
    __shared__ float Qi_[16][16][17]; // [node chunk of 16][column][k]  Qsub values
    const int c = blockIdx.y, r = a.r, RP = a.RP, n = a.n, N = a.N;
    const int cl = threadIdx.x / RP, k = threadIdx.x % RP;
    const int col = blockIdx.x * 16 + cl;
    const bool precise = a.gate && *a.gate != 0;
    const double* Tb = a.T + (size_t)c * r * r;
    for (int e = threadIdx.x; e < r * r; e += blockDim.x) Ts[e] = Tb[e];
    for (int e = threadIdx.x; e < RP * RP; e += blockDim.x) Ta[e] = a.Tacc[(size_t)c * RP * RP + e];
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
        Qi_[i & 15][cl][k] = (col < n && k < r) ? qv : 0.f;   // kept until Q' is known (N <= 16)
        mean += (double)qv;
    }
    float qm = (float)(mean / (double)N);
    if (col < n) {
        if (k < r) a.Qmean[((size_t)c * n + col) * r + k] = qm;
        if (a.sub_is_mean) a.Qsub[((size_t)c * n + col) * RP + k] = (k < r) ? qm : 0.f;
    }
    // Q' = Q Tacc (upper triangular): needs the whole row of Q
    __syncthreads();
    Ws[cl][k] = (col < n && k < r) ? qm : 0.f;
    __syncthreads();
    float qp = 0.f;
    for (int j = 0; j <= k; ++j) qp = fmaf(Ws[cl][j], Ta[j * RP + k], qp);
    if (!(col < n && k < r)) qp = 0.f;
    if (col < n) a.Qpad[((size_t)c * n + col) * RP + k] = qp;
    Qs_[cl][k] = qp;
    __syncthreads();
    // this block's share of C'[j][k] = (1/Nsub) sum_i sum_col Qsub_i[col][j] Q'[col][k]:
    // thread (cl, k) with cl < RP takes entry (j = cl, k).  Needs N <= 16 (the fused plan guarantees it).
    if (cl < RP) {
        const int j = cl;
        double s = 0.0;
        if (a.sub_is_mean) {
            for (int cc = 0; cc < 16; ++cc) s = fma((double)Ws[cc][j], (double)Qs_[cc][k], s);
        } else {
            for (int i = 0; i < N; ++i)
                for (int cc = 0; cc < 16; ++cc) s = fma((double)Qi_[i][cc][j], (double)Qs_[cc][k], s);
            s /= (double)N;
        }
        a.Cpart[(((size_t)c * gridDim.x + blockIdx.x) * RP + j) * RP + k] = s;
    }
}

// C' = sum of the per-block shares (fixed order), float32 [count][RP][RP].  grid: count, RP*RP threads.
__global__ void k_sum_c(const double* Cpart, float* Cmat, int nparts, int RP) {
    const int c = blockIdx.x, e = threadIdx.x;
    if (e >= RP * RP) return;
    double s = 0.0;
    for (int p = 0; p < nparts; ++p) s += Cpart[((size_t)c * nparts + p) * RP * RP + e];
    Cmat[(size_t)c * RP * RP + e] = (float)s;
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
