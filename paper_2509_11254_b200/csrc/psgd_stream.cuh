// Single-pass SSP-Comp step for up to 16 columns, pipelined through the L2 cache.
//
// The iteration has two global dependencies: P~ needs every row of every node before the
// back-projection Q_i = Delta_i^T P~ can start, and the residual needs Q_i.  As in the cluster kernel
// (psgd_fused.cuh) both are removed algebraically: the residual of the previous step is never stored
// (the buffer keeps Delta_{t-1}; e_t = Delta_{t-1} - P~_{t-1} Qsub_i^T is rebuilt from the small factors,
// Algorithm 2 last line folded into Eq. (7a)), and because P~ = P T for an upper-triangular T,
// Q_i = Delta_i^T P~ = (Delta_i^T P) T, so the back-projection of a row block only needs that row block's
// un-orthogonalised P (k_finish_p / k_finish_q apply T afterwards to the small matrices).
//
// What is new here is where the tile waits between its two uses: in the L2 cache.  One persistent CTA per
// multiprocessor runs two independent roles that meet only through flags in global memory:
//   * projection role (2 or 3 independent groups of 4 warps).  Work unit: 32 rows x up to 512 columns of one node, walked in tiles of 64 columns
//     that 16-byte cp.async copies stage in padded shared memory (G, the stored Delta, and the matching rows of Q'
//     and Qsub_i), two tiles in flight per group across unit borders.  A lane owns rows l and l + 16 (l = lane % 16), a half warp 8 columns: a thread forms
//         Delta_t = g + (Delta_{t-1} - P~_{t-1}[row,:] Qsub_i[cols,:]^T)
//     accumulates its row of Delta_t Q' in registers, and the tile is stored back with coalesced 128-bit stores.
//     A unit ends with its 32 x RP partial product in global memory and a counter increment; the group that completes
//     a 32-row block (all nodes, all column splits) sums the partials in a fixed order (node mean, All-Reduce Mean
//     of Algorithm 1), writes P' = P of the block and its Gram partial, and raises the block's ready flag.
//   * back-projection role (1 or 2 workers of 4 warps).  A worker owns (node, 256 columns, every KC-th group of 128 rows)
//     and keeps W_i = Delta_i^T P' for those columns in registers.  It waits for the group's four ready flags and
//     then reads the rows of Delta_t back -- a few microseconds after they were written, i.e. from L2, not from
//     HBM -- through a private cp.async ring (8 rows in flight per thread).
// So HBM sees 12 bytes per element (read G, read Delta_{t-1}, write Delta_t) whatever the number of columns,
// and neither role ever waits for the other inside a CTA.  The projection role never waits on a flag, so the
// kernel cannot deadlock as long as all CTAs are resident (cooperative launch).  Sums are formed in a fixed
// order (bit-reproducible).  The flag waits are bounded in time; one that runs out sets PSGD_W_TIMEOUT and the
// kernel carries on to its end.
#pragma once
#include "psgd_fused.cuh"

namespace psgd {

constexpr int SS_ROWS = 32;                 // rows of a projection unit = one row block (a lane owns rows l and l + 16, l = lane % 16)
constexpr int SS_GROUP = 4;                 // row blocks per back-projection group (128 rows)
constexpr int SS_TCOLS = 64;                // columns of a tile (256-byte row pieces: narrower ones cost DRAM efficiency)
constexpr int SS_PITCH = SS_TCOLS + 4;      // padded row pitch in floats: conflict-free 128-bit reads down a column of rows
constexpr int SS_MAXTPU = 8;                // tiles per unit at most (512 columns)
constexpr int SS_WPG = 4;                   // warps of a projection group
constexpr int SS_NST = 3;                   // stages of a group's ring
constexpr int SS_THREADS = 512;             // NG projection groups of 4 warps, 4 - NG back-projection workers of 4 warps
constexpr int SS_BCOLS = 256;               // columns per back-projection worker
constexpr int SS_BDEPTH = 8;                // rows in flight per back-projection thread

struct StreamArgs {
    const float* G;      // [count][N][m][n]   gradients
    float* Mbuf;         // [count][N][m][n]   in: Delta_{t-1} (e_t if !PENDING); out: Delta_t
    const float* Qpad;   // [count][n][RP]     Q' = Q_{t-1} T (preconditioned), rows padded to RP
    const float* Qsub;   // [count][N or 1][n][RP]  factor the pending residual subtracts  (PENDING only)
    const float* Ppad;   // [count][m][RP]     P~_{t-1}                                   (PENDING only)
    float* Ppart;        // [count][nrb][N][csplit][32][RP]  per-unit partial products
    float* Pout;         // [count][m][RP]     P' (node mean of Delta_t Q')
    float* Wpart;        // [count][2 KC][N][n][RP]  partial W_i = Delta_i^T P' per (row slot, row parity)
    double* gram;        // [count][nrb][r][r] partial P'^T P'
    unsigned* acnt;      // [count][nrb]       units finished per row block (zero at launch)
    unsigned* ready;     // [count][nrb]       1 once P' of the row block is in Pout (zero at launch)
    int* flags;          // device status word
    int m, n, r, N, count, nrb, ngrp, tpu, csplit, KC, CB;
    int qsub_per_node;   // 1: Qsub [count][N][n][RP], 0: [count][n][RP] (node-averaged factor)
};

template <int RP>
__host__ __device__ constexpr int stream_stage_floats() {
    return 2 * SS_ROWS * SS_PITCH + 2 * SS_TCOLS * RP + SS_ROWS * RP;   // G tile, Delta tile, Q' rows, Qsub rows, P~_{t-1} rows
}
// Projection groups per CTA: three where shared memory allows (the role is bound by instruction issue and latency, the
// back-projection role has time to spare), else two.
template <int RP>
__host__ __device__ constexpr int stream_groups() { return RP >= 16 ? 2 : 3; }
template <int RP>
__host__ __device__ constexpr size_t stream_smem_bytes() {
    return (size_t)stream_groups<RP>() * SS_NST * stream_stage_floats<RP>() * 4
         + (size_t)(4 - stream_groups<RP>()) * SS_GROUP * SS_ROWS * RP * 4          // P' rows of the back-projection workers
         + (size_t)(4 - stream_groups<RP>()) * SS_BDEPTH * 128 * 16                 // their cp.async rings
         + 64;                                                                      // role mailboxes
}

__device__ __forceinline__ void cp_async16_hint(unsigned smem_dst, const void* gmem, unsigned long long policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(smem_dst), "l"(gmem), "l"(policy) : "memory");
}
__device__ __forceinline__ void cp_async16_zfill_hint(unsigned smem_dst, const void* gmem, int src_bytes, unsigned long long policy) {
    asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;\n" ::"r"(smem_dst), "l"(gmem), "r"(src_bytes), "l"(policy) : "memory");
}
__device__ __forceinline__ f2p add2(f2p a, f2p b) {
    f2p d;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f2p sub2(f2p a, f2p b) {
    f2p d;
    asm("sub.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void named_barrier(int id, int threads) {
    asm volatile("bar.sync %0, %1;\n" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;\n" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;\n" : "=l"(t));
    return t;
}

template <int RP, bool PENDING>
__global__ void __launch_bounds__(SS_THREADS, 1) k_stream_step(StreamArgs a) {
    constexpr int STAGE = stream_stage_floats<RP>();
    extern __shared__ __align__(16) float ss_smem[];
    float* ring = ss_smem;
    constexpr int SS_NG = stream_groups<RP>(), SS_NBW = 4 - SS_NG, SS_A_THREADS = SS_NG * SS_WPG * 32;
    float* sPb = ring + (size_t)SS_NG * SS_NST * STAGE;                // [NBW][128][RP]
    unsigned char* brings = reinterpret_cast<unsigned char*>(sPb + SS_NBW * SS_GROUP * SS_ROWS * RP);   // [NBW][SS_BDEPTH][128] x 16 bytes
    int* mail = reinterpret_cast<int*>(brings + (size_t)SS_NBW * SS_BDEPTH * 128 * 16);   // [group]: this unit completed its row block; [4 + worker]: the worker gave up waiting

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Gd = gridDim.x, cta = blockIdx.x;
    const int upm = a.nrb * a.N * a.csplit;                  // units per matrix
    const int U = a.count * upm;
    const unsigned units_per_rb = (unsigned)(a.N * a.csplit);
    const int n = a.n, m = a.m;

    if (tid < 8) mail[tid] = 0;
    __syncthreads();
#ifdef PSGD_STREAM_TIMING
    if (tid == 0) atomicMax(reinterpret_cast<unsigned long long*>(a.flags + 16), ~global_ns());
#endif
    unsigned long long pol_first;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol_first));

    if (warp < SS_A_THREADS / 32) {
        // =====================================================================================
        // projection role: SS_NG independent groups of SS_WPG warps, each with its own units, ring and barrier, so that one
        // group's barrier and shared-memory latencies are covered by the other's arithmetic
        // =====================================================================================
        constexpr int GT = SS_WPG * 32;                        // threads of a group
        constexpr int CPW = SS_TCOLS / SS_WPG;                 // columns of the tile per warp: 8 for each half warp
        constexpr int CPH = CPW / 2;
        constexpr int NCH = (SS_ROWS * SS_TCOLS / 4) / GT;     // 16-byte pieces of a tile per thread
        const int ga = warp / SS_WPG, gw = warp % SS_WPG, gt = tid - ga * GT;
        const int bar_id = 1 + ga;
        const int vcta = cta * SS_NG + ga, Gv = Gd * SS_NG;    // the group's place among all groups of the grid
        const int nmine = vcta < U ? (U - vcta + Gv - 1) / Gv : 0;   // its units: vcta, vcta + Gv, ...
        const int T = nmine * a.tpu;                           // its tiles
        float* gring = ring + (size_t)ga * SS_NST * STAGE;
        auto decode = [&](int lu, int& c, int& rb, int& node, int& sp) {   // unit (vcta + lu Gv) -> matrix, row block, node, column split
            const int u = vcta + lu * Gv;
            c = u / upm;
            int rem = u % upm;
            rb = rem / (a.N * a.csplit);
            rem %= a.N * a.csplit;
            node = rem / a.csplit;
            sp = rem % a.csplit;
        };
        constexpr int RPT = 2;                                 // rows per thread: every row of Q' / Qsub read from shared memory serves both
        const int hw = lane >> 4, l16 = lane & 15;            // half warp (which 8 of the warp's 16 columns), row within the half
        constexpr int RP2 = RP / 2;
        f2p acc2[RPT][RP2];              // running sums of Delta_t[row, :] Q', pairs of adjacent k
        f2p pp2[RPT][PENDING ? RP2 : 1]; // P~_{t-1}[row, :], pairs of adjacent k
        int c = 0, rb = 0, node = 0, sp = 0;

        // Per-thread constants of the tile copies: this thread moves NCH 16-byte pieces of each 32 x 64 tile (rows lr,
        // lr + 32 / NCH, ..., columns lc4 .. lc4 + 3) and its share of the Q' / Qsub rows.  The cursors below are advanced tile
        // by tile (64 columns to the right) and re-derived from the unit number only once per unit, so that the index
        // arithmetic does not compete with the sums for issue slots.
        constexpr int RSTEP = SS_ROWS / NCH;
        const int lr = gt / (SS_TCOLS / 4), lc4 = (gt % (SS_TCOLS / 4)) * 4;
        const unsigned dst0 = (unsigned)(lr * SS_PITCH + lc4) * 4;
        int l_lu = 0, l_kt = 0, l_st = 0, l_col = 0, l_row0 = 0;
        size_t l_g[NCH], l_q = 0, l_qs = 0, l_pp = 0;
        auto load_tile = [&]() {          // copies of the next tile in sequence
            if (l_kt == 0) {
                int lc, lrb, lnode, lsp;
                decode(l_lu, lc, lrb, lnode, lsp);
                const size_t mat = (size_t)lc * a.N + lnode;
                l_row0 = lrb * SS_ROWS;
                l_col = lsp * a.tpu * SS_TCOLS;
#pragma unroll
                for (int i = 0; i < NCH; ++i) l_g[i] = (mat * m + min(l_row0 + lr + i * RSTEP, m - 1)) * (size_t)n + l_col + lc4;
                l_q = ((size_t)lc * n + l_col) * RP;
                l_qs = ((a.qsub_per_node ? mat : (size_t)lc) * n + l_col) * RP;
                l_pp = ((size_t)lc * m + l_row0) * RP;
            }
            float* st = gring + (size_t)l_st * STAGE;
            const unsigned sa = smem_u32(st) + dst0, sb = sa + SS_ROWS * SS_PITCH * 4;
            const int ok = (l_col + lc4) < n ? 16 : 0;
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
                cp_async16_zfill_hint(sa + i * (RSTEP * SS_PITCH * 4), a.G + (ok ? l_g[i] : 0), ok, pol_first);
                cp_async16_zfill_hint(sb + i * (RSTEP * SS_PITCH * 4), a.Mbuf + (ok ? l_g[i] : 0), ok, pol_first);
                l_g[i] += SS_TCOLS;
            }
            // the 64 rows of Q' (and of Qsub_i) for these columns are one contiguous piece of 64 RP floats
#pragma unroll
            for (int ch = gt; ch < SS_TCOLS * RP / 4; ch += GT) {
                const int okq = (l_col + (ch * 4) / RP) < n ? 16 : 0;
                cp_async16(st + 2 * SS_ROWS * SS_PITCH + ch * 4, a.Qpad + (okq ? l_q + ch * 4 : 0), okq);
                if (PENDING) cp_async16(st + 2 * SS_ROWS * SS_PITCH + SS_TCOLS * RP + ch * 4, a.Qsub + (okq ? l_qs + ch * 4 : 0), okq);
            }
            if (PENDING && l_kt == 0) {     // first tile of a unit: the unit's rows of P~_{t-1}
#pragma unroll
                for (int ch = gt; ch < SS_ROWS * RP / 4; ch += GT) {
                    const int okp = (l_row0 + (ch * 4) / RP) < m ? 16 : 0;
                    cp_async16(st + 2 * SS_ROWS * SS_PITCH + 2 * SS_TCOLS * RP + ch * 4, a.Ppad + (okp ? l_pp + ch * 4 : 0), okp);
                }
            }
            l_q += SS_TCOLS * RP; l_qs += SS_TCOLS * RP; l_col += SS_TCOLS;
            if (++l_st == SS_NST) l_st = 0;
            if (++l_kt == a.tpu) { l_kt = 0; ++l_lu; }
        };

        for (int s = 0; s < SS_NST - 1; ++s) {
            if (s < T) load_tile();
            cp_async_commit();
        }
        int kt = 0, lu = 0, cst = 0, ccol = 0;        // compute cursor: tile within the unit, unit, stage, first column of the tile
        size_t s_o = 0;                               // where this thread's first piece of the tile goes in Mbuf
        int s_rows = 0;                               // how many of its NCH pieces lie inside the matrix
        for (int t = 0; t < T; ++t) {
            cp_async_wait<SS_NST - 2>();
            named_barrier(bar_id, GT);             // tile t has landed for everyone; everyone is done with tile t - 1
            if (t + SS_NST - 1 < T) load_tile();
            cp_async_commit();
            float* st = gring + (size_t)cst * STAGE;
            float* sa = st + l16 * SS_PITCH;
            const float* sb = st + SS_ROWS * SS_PITCH + l16 * SS_PITCH;
            const float* sq = st + 2 * SS_ROWS * SS_PITCH;
            const float* sqs = sq + SS_TCOLS * RP;
            if (kt == 0) {
                decode(lu, c, rb, node, sp);
                ccol = sp * a.tpu * SS_TCOLS;
                const size_t mat = (size_t)c * a.N + node;
                const int row0 = rb * SS_ROWS;
                s_rows = row0 + lr < m ? min(NCH, (m - row0 - lr + RSTEP - 1) / RSTEP) : 0;
                s_o = (mat * m + row0 + lr) * (size_t)n + ccol + lc4;
#pragma unroll
                for (int rr = 0; rr < RPT; ++rr)
#pragma unroll
                    for (int k = 0; k < RP2; ++k) acc2[rr][k] = 0ull;
                if (PENDING) {
#pragma unroll
                    for (int rr = 0; rr < RPT; ++rr) {
                        const float* spp = sqs + SS_TCOLS * RP + (l16 + 16 * rr) * RP;
#pragma unroll
                        for (int k4 = 0; k4 < RP / 4; ++k4) {
                            const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(spp + 4 * k4);
                            pp2[rr][PENDING ? 2 * k4 : 0] = v.x;
                            pp2[rr][PENDING ? 2 * k4 + 1 : 0] = v.y;
                        }
                    }
                }
            }
            // The rows of Qsub and Q' are read from shared memory as warp-wide broadcasts, 128 bits at a time; such a read
            // occupies the shared-memory pipe for four cycles whatever it broadcasts, which is what bounds this role, so every
            // one of them is used for both rows of the thread (the two half warps read different rows of Q', which costs nothing more).
#pragma unroll
            for (int j4 = 0; j4 < CPH / 4; ++j4) {
                const int cb = gw * CPW + hw * CPH + j4 * 4;          // 4 columns of the tile
                float v[RPT][4];
#pragma unroll
                for (int rr = 0; rr < RPT; ++rr) {
                    const float4 g4 = *reinterpret_cast<const float4*>(sa + 16 * rr * SS_PITCH + cb);
                    const float4 d4 = *reinterpret_cast<const float4*>(sb + 16 * rr * SS_PITCH + cb);
                    v[rr][0] = d4.x; v[rr][1] = d4.y; v[rr][2] = d4.z; v[rr][3] = d4.w;      // (the stored Delta for now)
                    if (!PENDING) { v[rr][0] += g4.x; v[rr][1] += g4.y; v[rr][2] += g4.z; v[rr][3] += g4.w; }
                }
                if (PENDING) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const float* qs = sqs + (cb + j) * RP;
                        f2p cs2[RPT];
#pragma unroll
                        for (int rr = 0; rr < RPT; ++rr) cs2[rr] = 0ull;
#pragma unroll
                        for (int k4 = 0; k4 < RP / 4; ++k4) {
                            const ulonglong2 q2 = *reinterpret_cast<const ulonglong2*>(qs + 4 * k4);
#pragma unroll
                            for (int rr = 0; rr < RPT; ++rr) {
                                cs2[rr] = ffma2(pp2[rr][PENDING ? 2 * k4 : 0], q2.x, cs2[rr]);
                                cs2[rr] = ffma2(pp2[rr][PENDING ? 2 * k4 + 1 : 0], q2.y, cs2[rr]);
                            }
                        }
#pragma unroll
                        for (int rr = 0; rr < RPT; ++rr) {
                            const float2 cc = unpack2(cs2[rr]);
                            v[rr][j] -= cc.x + cc.y;
                        }
                    }
#pragma unroll
                    for (int rr = 0; rr < RPT; ++rr) {
                        const float4 g4 = *reinterpret_cast<const float4*>(sa + 16 * rr * SS_PITCH + cb);
                        v[rr][0] += g4.x; v[rr][1] += g4.y; v[rr][2] += g4.z; v[rr][3] += g4.w;
                    }
                }
#pragma unroll
                for (int rr = 0; rr < RPT; ++rr)
                    *reinterpret_cast<float4*>(sa + 16 * rr * SS_PITCH + cb) = make_float4(v[rr][0], v[rr][1], v[rr][2], v[rr][3]);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float* q = sq + (cb + j) * RP;
                    f2p vd[RPT];
#pragma unroll
                    for (int rr = 0; rr < RPT; ++rr) vd[rr] = pack2(v[rr][j], v[rr][j]);
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const ulonglong2 q2 = *reinterpret_cast<const ulonglong2*>(q + 4 * k4);
#pragma unroll
                        for (int rr = 0; rr < RPT; ++rr) {
                            acc2[rr][2 * k4] = ffma2(vd[rr], q2.x, acc2[rr][2 * k4]);
                            acc2[rr][2 * k4 + 1] = ffma2(vd[rr], q2.y, acc2[rr][2 * k4 + 1]);
                        }
                    }
                }
            }
            named_barrier(bar_id, GT);             // the tile of Delta_t is complete in shared memory
            if (ccol + lc4 < n) {
#pragma unroll
                for (int i = 0; i < NCH; ++i)
                    if (i < s_rows)
                        *reinterpret_cast<float4*>(a.Mbuf + s_o + (size_t)i * RSTEP * n) =
                            *reinterpret_cast<const float4*>(st + (lr + i * RSTEP) * SS_PITCH + lc4);
            }
            s_o += SS_TCOLS; ccol += SS_TCOLS;
            if (++cst == SS_NST) cst = 0;
            const bool unit_end = (kt == a.tpu - 1);
            if (++kt == a.tpu) { kt = 0; ++lu; }
            if (unit_end) {
                // ---- unit done: the half warps' sums in a fixed order -> the unit's 32 x RP partial product ----
                // (scratch [2 SS_WPG][32][RP], one slice per half warp: the stage just stored, which the next copies only reach after the next barrier)
                float* gred = st;
                named_barrier(bar_id, GT);         // everyone has read its pieces of the tile
#pragma unroll
                for (int rr = 0; rr < RPT; ++rr)
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const float2 x0 = unpack2(acc2[rr][2 * k4]), x1 = unpack2(acc2[rr][2 * k4 + 1]);
                        *reinterpret_cast<float4*>(gred + ((gw * 2 + hw) * SS_ROWS + l16 + 16 * rr) * RP + 4 * k4) = make_float4(x0.x, x0.y, x1.x, x1.y);
                    }
                named_barrier(bar_id, GT);
                for (int e4 = gt; e4 < SS_ROWS * RP / 4; e4 += GT) {
                    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int w = 0; w < 2 * SS_WPG; ++w) {
                        const float4 x = reinterpret_cast<const float4*>(gred + w * SS_ROWS * RP)[e4];
                        s4.x += x.x; s4.y += x.y; s4.z += x.z; s4.w += x.w;
                    }
                    float* out = a.Ppart + ((((size_t)c * a.nrb + rb) * a.N + node) * a.csplit + sp) * (SS_ROWS * RP);
                    reinterpret_cast<float4*>(out)[e4] = s4;
                }
                __threadfence();                   // the tile stores and the partial product, before the counter
                named_barrier(bar_id, GT);
                if (gt == 0) {
                    const unsigned old = atomicAdd(a.acnt + (size_t)c * a.nrb + rb, 1u);
                    mail[ga] = (old + 1u == units_per_rb) ? 1 : 0;
                }
                named_barrier(bar_id, GT);
                if (mail[ga]) {
                    // ---- this unit completed its row block: node mean of the partials (fixed order: node, then column split),
                    //      P' rows, Gram partial, ready flag ----
                    __threadfence();
                    const float* pb = a.Ppart + ((size_t)c * a.nrb + rb) * units_per_rb * (SS_ROWS * RP);
                    const int np = (int)units_per_rb;
                    const float nf = (float)a.N;
                    named_barrier(bar_id, GT);      // (the scratch is about to be overwritten with P')
                    for (int e4 = gt; e4 < SS_ROWS * RP / 4; e4 += GT) {
                        float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
                        int p = 0;
                        for (; p + 8 <= np; p += 8) {
                            float4 x[8];
#pragma unroll
                            for (int q = 0; q < 8; ++q) x[q] = __ldcg(reinterpret_cast<const float4*>(pb + (size_t)(p + q) * (SS_ROWS * RP)) + e4);
#pragma unroll
                            for (int q = 0; q < 8; ++q) { s4.x += x[q].x; s4.y += x[q].y; s4.z += x[q].z; s4.w += x[q].w; }
                        }
                        for (; p < np; ++p) {
                            const float4 x = __ldcg(reinterpret_cast<const float4*>(pb + (size_t)p * (SS_ROWS * RP)) + e4);
                            s4.x += x.x; s4.y += x.y; s4.z += x.z; s4.w += x.w;
                        }
                        const int row = rb * SS_ROWS + (e4 * 4) / RP;
                        if (row < m) {
                            s4.x /= nf; s4.y /= nf; s4.z /= nf; s4.w /= nf;
                            reinterpret_cast<float4*>(a.Pout + ((size_t)c * m + (size_t)rb * SS_ROWS) * RP)[e4] = s4;
                        } else {
                            s4 = make_float4(0.f, 0.f, 0.f, 0.f);     // (rows past the end were computed on a repeated last row)
                        }
                        reinterpret_cast<float4*>(gred)[e4] = s4;
                    }
                    named_barrier(bar_id, GT);
                    for (int e = gt; e < a.r * a.r; e += GT) {
                        const int ea = e / a.r, eb = e % a.r;
                        double g = 0.0;
                        for (int rr = 0; rr < SS_ROWS; ++rr) g = fma((double)gred[rr * RP + ea], (double)gred[rr * RP + eb], g);
                        a.gram[(((size_t)c * a.nrb + rb) * a.r + ea) * a.r + eb] = g;
                    }
                    __threadfence();
                    named_barrier(bar_id, GT);
                    if (gt == 0) st_release_u32(a.ready + (size_t)c * a.nrb + rb, 1u);
                }
            }
        }
        cp_async_wait<0>();
#ifdef PSGD_STREAM_TIMING
        if (gt == 0) atomicMax(reinterpret_cast<unsigned long long*>(a.flags + 18), global_ns());
#endif
    } else {
        // =====================================================================================
        // back-projection role
        // =====================================================================================
        const int w = (warp - SS_A_THREADS / 32) >> 2;          // worker of this CTA
        const int bt = tid - SS_A_THREADS - w * 128;            // thread of the worker
        const int tx = bt & 63, g = bt >> 6;                    // 4 columns, row parity
        constexpr int GR = SS_GROUP * SS_ROWS;                  // rows of a group
        float* Ps = sPb + w * GR * RP;                          // [128][RP]
        unsigned char* bring = brings + (size_t)w * (SS_BDEPTH * 128 * 16);
        const unsigned bslot = smem_u32(bring) + (unsigned)bt * 16;
        const unsigned char* bslot_g = bring + bt * 16;
        const int NW = SS_NBW * Gd, wk = SS_NBW * cta + w;
        const int ipm = a.KC * a.N * a.CB;                      // items per matrix
        const int nitems = a.count * ipm;
        for (int item = wk; item < nitems; item += NW) {
            const int c = item / ipm;
            int rem = item % ipm;
            const int slot = rem / (a.N * a.CB);
            rem %= a.N * a.CB;
            const int node = rem / a.CB, cb = rem % a.CB;
            const int col = cb * SS_BCOLS + tx * 4;
            const bool colok = col < n;
            const float* Mb = a.Mbuf + ((size_t)c * a.N + node) * (size_t)m * n + col;
            constexpr int RP2 = RP / 2;
            f2p wacc[4][RP2];    // W[col + j][k], pairs of adjacent k
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int k = 0; k < RP2; ++k) wacc[j][k] = 0ull;
            for (int grp = slot; grp < a.ngrp; grp += a.KC) {
                if (bt == 0 && !mail[4 + w]) {
                    const unsigned long long t0 = global_ns();
                    for (int rb = grp * SS_GROUP; rb < min(a.nrb, (grp + 1) * SS_GROUP); ++rb) {
                        const unsigned* f = a.ready + (size_t)c * a.nrb + rb;
                        while (ld_acquire_u32(f) == 0u) {
                            if (global_ns() - t0 > 2000000000ull) { mail[4 + w] = 1; atomicOr(a.flags, FU_W_TIMEOUT); break; }
                            __nanosleep(100);
                        }
                        if (mail[4 + w]) break;
                    }
                }
                named_barrier(8 + w, 128);
                // P' rows of the group
                const int row0 = grp * GR;
                for (int e4 = bt; e4 < GR * RP / 4; e4 += 128) {
                    const int row = row0 + (e4 * 4) / RP;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (row < m) v = __ldcg(reinterpret_cast<const float4*>(a.Pout + ((size_t)c * m + row0) * RP) + e4);
                    reinterpret_cast<float4*>(Ps)[e4] = v;
                }
                named_barrier(8 + w, 128);
                const int nrows = max(0, min((min(m, row0 + GR) - row0 - g + 1) / 2, GR / 2));   // this thread's rows inside the matrix
                // This thread's rows of the group (row parity g), 4 columns each, come through a private ring of SS_BDEPTH
                // 16-byte slots in shared memory filled by cp.async: SS_BDEPTH rows are in flight per thread without
                // holding registers, which is what hides the L2 latency; nobody else touches the slots, so no barrier.
                const float* src = Mb + (size_t)(row0 + g) * n;
                auto fetch = [&](int rr) {      // row index rr of this thread -> slot rr % SS_BDEPTH
                    if (rr < nrows && colok) cp_async16_hint(bslot + (rr % SS_BDEPTH) * (128 * 16), src + (size_t)rr * 2 * n, pol_first);
                    cp_async_commit();
                };
#pragma unroll 1
                for (int rr = 0; rr < SS_BDEPTH; ++rr) fetch(rr);
                if (colok) {
#pragma unroll 1
                    for (int rr = 0; rr < nrows; ++rr) {
                        cp_async_wait<SS_BDEPTH - 1>();
                        const float4 v = *reinterpret_cast<const float4*>(bslot_g + (rr % SS_BDEPTH) * (128 * 16));
                        fetch(rr + SS_BDEPTH);
                        const float* pr = Ps + (g + 2 * rr) * RP;
                        const f2p vd[4] = {pack2(v.x, v.x), pack2(v.y, v.y), pack2(v.z, v.z), pack2(v.w, v.w)};
#pragma unroll
                        for (int k4 = 0; k4 < RP / 4; ++k4) {
                            const ulonglong2 p4 = *reinterpret_cast<const ulonglong2*>(pr + 4 * k4);
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                wacc[j][2 * k4] = ffma2(vd[j], p4.x, wacc[j][2 * k4]);
                                wacc[j][2 * k4 + 1] = ffma2(vd[j], p4.y, wacc[j][2 * k4 + 1]);
                            }
                        }
                    }
                }
                cp_async_wait<0>();
            }
#ifdef PSGD_STREAM_TIMING
            if (bt == 0) atomicMax(reinterpret_cast<unsigned long long*>(a.flags + 20), global_ns());
#endif
            // this worker's partial W for (row slot, row parity)
            if (colok) {
                float* wo = a.Wpart + ((((size_t)c * (2 * a.KC) + 2 * slot + g) * a.N + node) * n + col) * RP;
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int k4 = 0; k4 < RP / 4; ++k4) {
                        const float2 x0 = unpack2(wacc[j][2 * k4]), x1 = unpack2(wacc[j][2 * k4 + 1]);
                        *reinterpret_cast<float4*>(wo + (size_t)j * RP + 4 * k4) = make_float4(x0.x, x0.y, x1.x, x1.y);
                    }
            }
        }
    }
}

}  // namespace psgd
