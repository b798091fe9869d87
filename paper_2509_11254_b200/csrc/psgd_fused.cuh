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
// owns a column slice of WC columns.  The CTA's 16 warps are split into two roles with their
// own register budgets (setmaxnreg):
//   * 8 projection warps: G and the stored Delta arrive as TMA tiles (cp.async.bulk.tensor,
//     zero fill beyond the matrix edges) in a ring of shared-memory stages tracked by
//     mbarriers; the warps take turns issuing the copies, form S, keep it in a double-buffered
//     shared-memory tile, accumulate S Q' and send the 8 x r partial sums of P to every CTA
//     of the cluster (st.async into the peers' shared memory, counted by their mbarriers);
//   * 8 back-projection warps: one block behind, they finish P' of a block, apply the
//     correction to the tile, accumulate W in registers and write Delta_t to HBM.
// The two roles meet only through mbarriers (tile written / tile free), so the latency of
// the cluster exchange and of either role is covered by the other.
// Float sums are formed in a fixed order everywhere (bit-reproducible results).  Every
// mbarrier wait is bounded; a wait that runs out sets PSGD_W_TIMEOUT in the status word and
// the kernel carries on to its end.
#pragma once
#include <cooperative_groups.h>
#include <cuda.h>

#include "psgd_kernels.cuh"

namespace psgd {
namespace cg = cooperative_groups;

constexpr int FU_THREADS = 512;     // 8 projection warps + 8 back-projection warps
constexpr int FU_ROLE = 256;        // threads per role
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
    static constexpr int BW = WC >= 256 ? 256 : WC;      // columns of one TMA tile
    static constexpr int NBX = WC / BW;                  // TMA tiles per array and stage
    static constexpr int CPL = WC >= 256 ? 2 : 1;        // columns per lane in the projection role
    static constexpr int NCG = WC / (32 * CPL);          // column groups of a stage (one warp each)
    static constexpr int NRG = 8 / NCG;                  // row groups of a stage
    static constexpr int RS = FU_RG * NRG;               // rows of a stage
    static constexpr int NRC = FU_R / RS;                // stages (row chunks) per node and block
    static constexpr int NST = WC >= 256 ? 5 : 8;        // ring depth
    static constexpr int TPN = WC / 8;                   // back-projection threads per node
    static constexpr int STAGE_FLOATS = 2 * RS * WC;     // G rows, then stored-Delta rows; each array as NBX tiles [RS][BW]
    static constexpr int NBAR = 2 * NST + 6;             // full/empty per stage, 2 x (received, tile written, tile free)
};

template <int RP, int WC>
__host__ __device__ inline size_t fused_smem_bytes(int N) {
    using Ge = FusedGeom<WC>;
    size_t fl = (size_t)2 * N * FU_R * WC            // S tile, double-buffered
              + (size_t)Ge::NST * Ge::STAGE_FLOATS   // ring
              + (size_t)2 * 2 * Ge::NCG * 32         // per-warp partial sums of P
              + (size_t)2 * FU_MAXCS * FU_R * RP     // partial sums received from the cluster
              + (size_t)3 * 2 * FU_R * RP            // P' rows, P' rows with swapped pairs, -P~_{t-1} rows
              + (size_t)RP * RP;                     // C'
    return fl * 4 + (size_t)Ge::NBAR * 8 + 128;      // + alignment slack for the TMA destinations
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
#ifdef PSGD_MBAR_TEST_WAIT
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
#else
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
#endif
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
// For a role played by a single thread whose barrier has usually completed already: a non-blocking test first.
__device__ __forceinline__ void mbar_wait_ready(unsigned bar, unsigned parity, int* flags, bool& dead) {
    unsigned ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (!ok) mbar_wait(bar, parity, flags, dead);
}
// The same wait for a whole warp (all 32 lanes must call it): lane 0 polls, pausing between polls, so that a waiting
// warp puts one request at a time on the barrier instead of 32 (many warps polling at full rate slow down every other
// barrier operation of the CTA, the single MMA-issuing thread's first of all); once the phase has completed every lane
// observes it itself with one more try_wait, which returns at once and gives that lane its own acquire.
__device__ __forceinline__ void mbar_wait_warp(unsigned bar, unsigned parity, int* flags, bool& dead) {
    if (dead) return;                        // (uniform across the warp: set from lane 0 below)
    int gave_up = 0;
    if ((threadIdx.x & 31) == 0) {
        bool ok = false;
        for (unsigned it = 0; it < FU_WAIT_LIMIT && !ok; ++it) {
            ok = mbar_try_wait(bar, parity);
            if (!ok) __nanosleep(40);
        }
        if (!ok) { gave_up = 1; atomicOr(flags, FU_W_TIMEOUT); }
    }
    gave_up = __shfl_sync(0xffffffffu, gave_up, 0);
    if (gave_up) { dead = true; return; }
#ifndef PSGD_MBAR_NO_REWAIT
    (void)mbar_try_wait(bar, parity);
#endif
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

// A float delivered to a peer CTA's shared memory; the peer's mbarrier counts the 4 bytes.
__device__ __forceinline__ void st_async_cluster_f32(unsigned local_addr, unsigned local_bar, unsigned rank, float v) {
    unsigned raddr, rbar;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(raddr) : "r"(local_addr), "r"(rank));
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;\n" : "=r"(rbar) : "r"(local_bar), "r"(rank));
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];\n"
                 ::"r"(raddr), "r"(__float_as_uint(v)), "r"(rbar) : "memory");
}

// The same over each half warp (16 lanes) of NV in {8, 16} per-lane values: on return lane l holds the total of
// value index l & 15 (NV == 16) or (l & 15) >> 1 (NV == 8) of its half in v[0].
template <int NV>
__device__ __forceinline__ void butterfly_reduce16(float (&v)[NV], int lane) {
#pragma unroll
    for (int o = 8, cnt = NV; cnt > 1; o >>= 1, cnt >>= 1) {
        const bool up = (lane & o) != 0;
#pragma unroll
        for (int j = 0; j < cnt / 2; ++j) {
            float send = up ? v[j] : v[j + cnt / 2];
            float keep = up ? v[j + cnt / 2] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    if (NV == 8) v[0] += __shfl_xor_sync(0xffffffffu, v[0], 1);
}

__device__ __forceinline__ void role_barrier(int id) {   // barrier among the 256 threads of one role
    asm volatile("bar.sync %0, 256;\n" ::"r"(id) : "memory");
}

template <int RP, int WC, bool PENDING, bool GBF = false>   // GBF: the gradient tiles are bfloat16 (half the bytes of their slot)
__global__ void __launch_bounds__(FU_THREADS, 1)
k_fused_step(const __grid_constant__ CUtensorMap tmG, const __grid_constant__ CUtensorMap tmM, FusedArgs a) {
    using Ge = FusedGeom<WC>;
    constexpr int BW = Ge::BW, NBX = Ge::NBX, CPL = Ge::CPL, NCG = Ge::NCG, RS = Ge::RS, NRC = Ge::NRC, NST = Ge::NST, TPN = Ge::TPN;
    constexpr int PR = FU_R * RP;          // entries of one block of P
    constexpr int RP2 = RP / 2;
    constexpr unsigned STAGE_BYTES = Ge::STAGE_FLOATS * 4;
    constexpr unsigned BOX_BYTES = RS * BW * 4;

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
    float* ring = smem;                                        // [NST][2][NBX][RS][BW]   (128-byte aligned)
    float* tile = ring + (size_t)NST * Ge::STAGE_FLOATS;       // [2][N][8][WC]
    float* PpartW = tile + (size_t)2 * N * FU_R * WC;          // [2][2][NCG][32]
    float* Precv = PpartW + 2 * 2 * NCG * 32;                  // [2][FU_MAXCS][PR]
    float* Pb = Precv + 2 * FU_MAXCS * PR;                     // [2][PR]   P' rows
    float* Pbs = Pb + 2 * PR;                                  // [2][PR]   P' rows, neighbours (2k, 2k+1) swapped
    float* Ppn = Pbs + 2 * PR;                                 // [2][PR]   -P~_{t-1} rows
    float* Cm = Ppn + 2 * PR;                                  // [RP][RP]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(Cm + RP * RP);
    const unsigned bar_full = smem_u32(bars), bar_empty = bar_full + 8 * NST, bar_recv = bar_empty + 8 * NST;
    const unsigned bar_tfull = bar_recv + 16, bar_tfree = bar_tfull + 16;

    float* Mc = a.Mbuf + (size_t)c * N * m * n;

    // row blocks this cluster owns: slot, slot + KC, ...
    const int nb = (a.nblk > slot) ? (a.nblk - slot + a.KC - 1) / a.KC : 0;
    const int nstb = NRC * N;              // stages per block: row chunk outer, node inner
    const int T = nb * nstb;

    // ---- one-time set-up ----
    if (tid == 0) {
        for (int s = 0; s < NST; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, FU_ROLE / 32);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_recv + 8 * b, 1);
            mbar_init(bar_tfull + 8 * b, FU_ROLE / 32);
            mbar_init(bar_tfree + 8 * b, FU_ROLE / 32);
        }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (PENDING)
        for (int e = tid; e < RP * RP; e += FU_THREADS) Cm[e] = a.Cmat[(size_t)c * RP * RP + e];
    cluster.sync();   // every CTA's barriers exist before a peer sends to them
    bool dead = false;
    const f2p ZERO2 = 0ull;

    if (warp < FU_ROLE / 32) {
        // =====================================================================================
        // projection role
        // =====================================================================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 88;\n");
        const float* Qc = a.Qpad + (size_t)c * n * RP;
        // warp -> (column group, row group) of a stage (fixed for the kernel).  Slices of >= 256 columns: a warp
        // tile is 4 rows x 64 columns, lane -> (2 of the 4 rows, 4 adjacent columns), so that a half warp
        // covers a row contiguously and only 16 values per lane have to be reduced over 16 lanes.
        // Slices of 128 columns: 4 rows x 32 columns, lane -> one column.
        constexpr bool WIDE = (CPL == 2);
        constexpr int LC = WIDE ? 4 : 1;             // columns per lane
        constexpr int LR = WIDE ? 2 : FU_RG;         // rows per lane
        const int cgp = warp % NCG, rgl = warp / NCG;
        const int hrow = WIDE ? (lane >> 4) : 0;     // which row pair of the warp tile
        const int acol = WIDE ? cgp * 64 + 4 * (lane & 15) : cgp * 32 + lane;   // first column within the slice
        const int abox = acol / BW, aboxcol = acol % BW;                    // TMA tile and column inside it
        f2p Qr[LC][RP2];         // rows of Q' for this lane's columns, pairs over k
#pragma unroll
        for (int j = 0; j < LC; ++j)
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                ulonglong2 v = make_ulonglong2(0ull, 0ull);
                if (acol + j < ncols) v = __ldg(reinterpret_cast<const ulonglong2*>(Qc + (size_t)(colbase + acol + j) * RP + 4 * k4));
                Qr[j][2 * k4] = v.x;
                Qr[j][2 * k4 + 1] = v.y;
            }

        // producer duty (taken in turn by the warps): 2 * NBX TMA tiles per stage.
        // State of the next stage to issue, advanced by every thread in step with the main loop.
        int p_bl = 0, p_rc = 0, p_i = 0, p_ss = 0, p_par = 1;   // p_par: parity of the slot's previous release
        auto issue_next = [&]() {      // called by one whole warp; the slot must have been released
            if (lane == 0) {
                const int row = (slot + p_bl * a.KC) * FU_R + p_rc * RS;
                const unsigned bar = bar_full + 8 * p_ss;
                const unsigned dst = smem_u32(ring + (size_t)p_ss * Ge::STAGE_FLOATS);
                mbar_expect_tx(bar, GBF ? STAGE_BYTES / 2 + STAGE_BYTES / 4 : STAGE_BYTES);
#pragma unroll
                for (int x = 0; x < NBX; ++x) {
                    tma_load_3d(dst + x * (GBF ? BOX_BYTES / 2 : BOX_BYTES), &tmG, colbase + x * BW, row, c * N + p_i, bar);
                    tma_load_3d(dst + STAGE_BYTES / 2 + x * BOX_BYTES, &tmM, colbase + x * BW, row, c * N + p_i, bar);
                }
            }
            __syncwarp();
        };
        auto advance_next = [&]() {
            if (++p_i == N) { p_i = 0; if (++p_rc == NRC) { p_rc = 0; ++p_bl; } }
            if (++p_ss == NST) { p_ss = 0; p_par ^= 1; }
        };
        // The ring runs NST - 2 stages ahead: the slot refilled at stage sg is the one released two stages
        // earlier, so the warp on duty practically never waits for a slower warp.
        for (int s = 0; s < NST - 2; ++s) {
            if (s < T && warp == 0) issue_next();
            advance_next();
        }

        f2p sacc[LR][RP2];
#pragma unroll
        for (int rr = 0; rr < LR; ++rr)
#pragma unroll
            for (int k = 0; k < RP2; ++k) sacc[rr][k] = ZERO2;
        int ss = 0, par = 0;                // ring slot and parity of the stage being consumed
        int sg = 0;
        for (int bl = 0; bl < nb; ++bl) {
            const int pbuf = bl & 1;
            // the tile buffer was last read by the back-projection of block bl - 2
            if (bl >= 2) mbar_wait(bar_tfree + 8 * pbuf, (unsigned)(((bl >> 1) - 1) & 1), a.flags, dead);
#pragma unroll 1
            for (int rc = 0; rc < NRC; ++rc) {
#pragma unroll 1
                for (int i = 0; i < N; ++i, ++sg) {
                    if (warp == (sg & 7)) {           // this warp's turn to refill the ring
                        if (sg + NST - 2 < T) {
                            if (sg > 1) mbar_wait(bar_empty + 8 * p_ss, (unsigned)p_par, a.flags, dead);
                            issue_next();
                        }
                    }
                    advance_next();

                    // ---- S = g + stored Delta -> tile; sacc += S Q' ----
                    mbar_wait(bar_full + 8 * ss, (unsigned)par, a.flags, dead);
                    const size_t tile_off = (size_t)abox * (RS * BW) + (size_t)(rgl * FU_RG + hrow * LR) * BW + aboxcol;
                    const float* sgp = ring + (size_t)ss * Ge::STAGE_FLOATS + tile_off;
                    const unsigned short* sgb = reinterpret_cast<const unsigned short*>(ring + (size_t)ss * Ge::STAGE_FLOATS) + tile_off;
                    const float* smp = sgp + RS * WC;
                    float* tp = tile + (((size_t)pbuf * N + i) * FU_R + rc * RS + rgl * FU_RG + hrow * LR) * WC + acol;
                    float sv[LR][LC];
#pragma unroll
                    for (int rr = 0; rr < LR; ++rr) {
                        if (WIDE) {
                            float4 g4;
                            if (GBF) {      // bfloat16 -> float32: its 16 bits are the upper half
                                const uint2 gb = *reinterpret_cast<const uint2*>(sgb + rr * BW);
                                g4 = make_float4(__uint_as_float(gb.x << 16), __uint_as_float(gb.x & 0xFFFF0000u),
                                                 __uint_as_float(gb.y << 16), __uint_as_float(gb.y & 0xFFFF0000u));
                            } else {
                                g4 = *reinterpret_cast<const float4*>(sgp + rr * BW);
                            }
                            const float4 m4 = *reinterpret_cast<const float4*>(smp + rr * BW);
                            sv[rr][0] = g4.x + m4.x; sv[rr][LC > 1 ? 1 : 0] = g4.y + m4.y;
                            sv[rr][LC > 2 ? 2 : 0] = g4.z + m4.z; sv[rr][LC > 3 ? 3 : 0] = g4.w + m4.w;
                        } else {
                            sv[rr][0] = (GBF ? __uint_as_float((unsigned)sgb[rr * BW] << 16) : sgp[rr * BW]) + smp[rr * BW];
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_empty + 8 * ss);   // the stage is in registers: release the slot
#pragma unroll
                    for (int rr = 0; rr < LR; ++rr) {
                        if (WIDE) *reinterpret_cast<float4*>(tp + rr * WC) = make_float4(sv[rr][0], sv[rr][LC > 1 ? 1 : 0], sv[rr][LC > 2 ? 2 : 0], sv[rr][LC > 3 ? 3 : 0]);
                        else tp[rr * WC] = sv[rr][0];
#pragma unroll
                        for (int j = 0; j < LC; ++j) {
                            const f2p sd = pack2(sv[rr][j], sv[rr][j]);
#pragma unroll
                            for (int k2 = 0; k2 < RP2; ++k2) sacc[rr][k2] = ffma2(sd, Qr[j][k2], sacc[rr][k2]);
                        }
                    }
                    if (++ss == NST) { ss = 0; par ^= 1; }

                    if (i == N - 1) {   // the row chunk is complete for every node: reduce over the warp's columns
                        constexpr int LV = LR * RP;      // values per lane
                        float v[LV];
#pragma unroll
                        for (int rr = 0; rr < LR; ++rr)
#pragma unroll
                            for (int k2 = 0; k2 < RP2; ++k2) {
                                const float2 u = unpack2(sacc[rr][k2]);
                                v[rr * RP + 2 * k2] = u.x;
                                v[rr * RP + 2 * k2 + 1] = u.y;
                                sacc[rr][k2] = ZERO2;
                            }
                        const int rgi = rc * Ge::NRG + rgl;     // row group within the block (0 or 1)
                        float* pw = PpartW + ((pbuf * 2 + rgi) * NCG + cgp) * 32;   // [row in group][k]
                        if (WIDE) {
                            butterfly_reduce16<LV>(v, lane);
                            if (LV == 16) pw[hrow * LV + (lane & 15)] = v[0];
                            else if ((lane & 1) == 0) pw[hrow * LV + ((lane & 15) >> 1)] = v[0];
                        } else {
                            butterfly_reduce<LV>(v, lane);
                            if (LV == 32 || (lane & 1) == 0) pw[LV == 32 ? lane : lane >> 1] = v[0];
                        }
                    }
                }
            }
            // block projected: the tile is complete; CTA sum of the partial P, sent to every CTA of the cluster
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tfull + 8 * pbuf);
            role_barrier(1);
            if (tid < PR) {
                const int rr = tid / RP, k = tid % RP;
                const int rgi = rr / FU_RG, j = (rr % FU_RG) * RP + k;
                float sum = 0.f;
#pragma unroll
                for (int g = 0; g < NCG; ++g) sum += PpartW[((pbuf * 2 + rgi) * NCG + g) * 32 + j];
                const unsigned dst = smem_u32(Precv + (pbuf * FU_MAXCS + q) * PR + tid);
                for (int qq = 0; qq < CS; ++qq) st_async_cluster_f32(dst, bar_recv + 8 * pbuf, (unsigned)qq, sum);
            }
        }
    } else {
        // =====================================================================================
        // back-projection role (one block behind the projection)
        // =====================================================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 168;\n");
        const int tb = tid - FU_ROLE;
        const float* Ppc = PENDING ? a.Ppad + (size_t)c * m * RP : nullptr;
        const float* Qsc = PENDING ? a.Qsub + (size_t)c * (a.qsub_node_stride ? N : 1) * n * RP : nullptr;
        // thread -> (node, 4 + 4 columns)
        const int bi = tb / TPN, tc = tb % TPN;
        const bool btask = bi < N;
        const int bc0 = 4 * tc, bc1 = WC / 2 + 4 * tc;
        const bool bok0 = btask && bc0 < ncols, bok1 = btask && bc1 < ncols;
        // W for 8 columns in "diagonal" pairs: wd[j2][k2][0] = {w[2j2][2k2], w[2j2+1][2k2+1]}, [1] = {w[2j2][2k2+1], w[2j2+1][2k2]}
        f2p wd[4][RP2][2];
        constexpr int QSN = PENDING ? 8 : 1;
        f2p qs[QSN][RP2];                      // Qsub rows of the 8 columns, pairs over k
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < RP2; ++k) { wd[j][k][0] = ZERO2; wd[j][k][1] = ZERO2; }
        if (PENDING) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = (j < 4 ? bc0 : bc1) + (j & 3);
#pragma unroll
                for (int k4 = 0; k4 < RP / 4; ++k4) {
                    ulonglong2 v = make_ulonglong2(0ull, 0ull);
                    if (btask && col < ncols)
                        v = __ldg(reinterpret_cast<const ulonglong2*>(Qsc + (size_t)bi * a.qsub_node_stride + (size_t)(colbase + col) * RP + 4 * k4));
                    qs[j % QSN][2 * k4] = v.x;
                    qs[j % QSN][2 * k4 + 1] = v.y;
                }
            }
        }
        double gacc = 0.0;   // rank 0, threads 64 .. 64 + r*r of the role: one entry of P'^T P'

        for (int bl = 0; bl < nb; ++bl) {
            const int pb = bl & 1;
            const int prow0 = (slot + bl * a.KC) * FU_R;
            const unsigned ph = (unsigned)((bl >> 1) & 1);
            float pprev = 0.f;
            if (PENDING && tb < PR) {
                const int rr = tb / RP;
                pprev = (prow0 + rr < m) ? __ldg(Ppc + (size_t)(prow0 + rr) * RP + tb % RP) : 0.f;
            }
            if (tb == 0) mbar_expect_tx(bar_recv + 8 * pb, (unsigned)(CS * PR * 4));
            if (PENDING && tb < PR) Ppn[pb * PR + tb] = -pprev;
            role_barrier(2);                      // -P~_{t-1} rows visible to the role
            // P' of the block: node mean of the cluster's partial sums, small-space correction.
            // Every thread waits for the sums itself (bounded), so no barrier precedes the reads.
            mbar_wait(bar_recv + 8 * pb, ph, a.flags, dead);
            if (tb < PR) {
                const int rr = tb / RP, k = tb % RP;
                float sum = 0.f;
                for (int qq = 0; qq < CS; ++qq) sum += Precv[(pb * FU_MAXCS + qq) * PR + tb];
                float v = sum / (float)N;
                if (PENDING) {
                    const float* pp = Ppn + pb * PR + rr * RP;
#pragma unroll
                    for (int j = 0; j < RP; ++j) v = fmaf(pp[j], Cm[j * RP + k], v);
                }
                if (prow0 + rr >= m) v = 0.f;
                Pb[pb * PR + tb] = v;
                Pbs[pb * PR + (tb ^ 1)] = v;
                if (q == 0 && prow0 + rr < m) a.Pout[((size_t)c * m + prow0 + rr) * RP + k] = v;
            }
            role_barrier(2);                      // P' rows visible to the role
            {
                const int t2 = tb - 64;
                if (q == 0 && t2 >= 0 && t2 < a.r * a.r) {
                    const int ga = t2 / a.r, gb = t2 % a.r;
#pragma unroll
                    for (int rr = 0; rr < FU_R; ++rr)
                        gacc = fma((double)Pb[pb * PR + rr * RP + ga], (double)Pb[pb * PR + rr * RP + gb], gacc);
                }
            }
            mbar_wait(bar_tfull + 8 * pb, ph, a.flags, dead);   // all of S of this block is in the tile
            if (btask) {
                // rows of the block: Delta = S - P~_{t-1} Qsub^T, W += Delta^T P', store Delta
#pragma unroll 1
                for (int rr = 0; rr < FU_R; ++rr) {
                    const float* tp = tile + (((size_t)pb * N + bi) * FU_R + rr) * WC;
                    const float4 v0 = *reinterpret_cast<const float4*>(tp + bc0);
                    const float4 v1 = *reinterpret_cast<const float4*>(tp + bc1);
                    float mvs[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                    if (PENDING) {
                        const float* pp = Ppn + pb * PR + rr * RP;
                        f2p pn2[RP2];
#pragma unroll
                        for (int k4 = 0; k4 < RP / 4; ++k4) {
                            const ulonglong2 p4 = *reinterpret_cast<const ulonglong2*>(pp + 4 * k4);
                            pn2[2 * k4] = p4.x;
                            pn2[2 * k4 + 1] = p4.y;
                        }
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            f2p acc = ffma2(pn2[0], qs[j % QSN][0], ZERO2);
#pragma unroll
                            for (int k2 = 1; k2 < RP2; ++k2) acc = ffma2(pn2[k2], qs[j % QSN][k2], acc);
                            const float2 u = unpack2(acc);
                            mvs[j] += u.x + u.y;
                        }
                    }
                    const float* pr = Pb + pb * PR + rr * RP;
                    const float* prs = Pbs + pb * PR + rr * RP;
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const ulonglong2 p4 = *reinterpret_cast<const ulonglong2*>(pr + 4 * k4);
                        const ulonglong2 s4 = *reinterpret_cast<const ulonglong2*>(prs + 4 * k4);
                        const f2p pk2[2] = {p4.x, p4.y};
                        const f2p pks2[2] = {s4.x, s4.y};
#pragma unroll
                        for (int j2 = 0; j2 < 4; ++j2) {
                            const f2p mp = pack2(mvs[2 * j2], mvs[2 * j2 + 1]);
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                wd[j2][2 * k4 + u][0] = ffma2(mp, pk2[u], wd[j2][2 * k4 + u][0]);
                                wd[j2][2 * k4 + u][1] = ffma2(mp, pks2[u], wd[j2][2 * k4 + u][1]);
                            }
                        }
                    }
                    if (prow0 + rr < m) {
                        float* go = Mc + ((size_t)bi * m + prow0 + rr) * n + colbase;
                        if (bok0) *reinterpret_cast<float4*>(go + bc0) = make_float4(mvs[0], mvs[1], mvs[2], mvs[3]);
                        if (bok1) *reinterpret_cast<float4*>(go + bc1) = make_float4(mvs[4], mvs[5], mvs[6], mvs[7]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_tfree + 8 * pb);   // the projection may overwrite this tile buffer
        }

        // ---- flush this cluster's partial W and Gram ----
        if (btask) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int col = (j < 4 ? bc0 : bc1) + (j & 3);
                if (col < ncols) {
                    float* wp = a.Wpart + ((((size_t)c * a.KC + slot) * N + bi) * n + colbase + col) * RP;
                    const int j2 = j >> 1, odd = j & 1;
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        // w[j][2k2] and w[j][2k2+1] out of the diagonal pairs
                        const float2 a0 = unpack2(wd[j2][2 * k4][0]), b0 = unpack2(wd[j2][2 * k4][1]);
                        const float2 a1 = unpack2(wd[j2][2 * k4 + 1][0]), b1 = unpack2(wd[j2][2 * k4 + 1][1]);
                        *reinterpret_cast<float4*>(wp + 4 * k4) = odd ? make_float4(b0.y, a0.y, b1.y, a1.y)
                                                                       : make_float4(a0.x, b0.x, a1.x, b1.x);
                    }
                }
            }
        }
        {
            const int t2 = tb - 64;
            if (q == 0 && t2 >= 0 && t2 < a.r * a.r) a.gram[((size_t)c * a.KC + slot) * a.r * a.r + t2] = gacc;
        }
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
