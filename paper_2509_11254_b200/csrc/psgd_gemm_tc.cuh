// Tensor-core contraction for the refresh (SVD-Comp of Algorithm 1, computed as a block
// subspace iteration):  C = A B^T  with A [M][K] and B [Nc][K] both row-major float32, i.e. both
// operands K-major.  The two products of one iteration have this form,
//     Y = Dbar Z      (A = Dbar  [m][n],  B = Z^T [l][n]),
//     Z = Dbar^T Y    (A = Dbar^T [n][m], B = Y^T [l][m]),
// once a transposed copy of the node mean Dbar is kept.
//
// sm_100 path: TMA loads 128-byte-swizzled tiles (128 x 32 floats of A, Ncp x 32 of B) into a
// 4-stage shared-memory ring; one thread issues tcgen05.mma (kind::tf32, M = 128, N = Ncp,
// K = 8 per instruction) with the accumulator in tensor memory; four warps read the
// accumulator back with tcgen05.ld and store it.  Inputs are read as TF32 (the low 13 mantissa
// bits of the float32 operands are ignored), which is why the refresh only runs its early
// sweeps here and finishes with float32 sweeps.  K is split over blockIdx.y; the partial
// products are summed in a fixed order by k_gemm_reduce.
// Every wait is bounded: a wait that runs out sets PSGD_W_TIMEOUT and the kernel carries on,
// frees its tensor memory and returns.
#pragma once
#include <cuda.h>

#include "psgd_fused.cuh"

namespace psgd {

constexpr int TC_BM = 128;       // rows of A per CTA (= UMMA M)
constexpr int TC_BK = 32;        // floats of K per stage (= one 128-byte swizzle row)
constexpr int TC_STAGES = 4;
constexpr int TC_THREADS = 192;  // warp 0: TMA, warp 1: MMA + tensor-memory owner, warps 2-5: epilogue
constexpr int TC_MAXN = 256;

struct GemmTcArgs {
    float* Cpart;     // [count][S][M][Ncp]
    int M, Ncp, K, S, kb_per_split;
    int* flags;
};

__host__ __device__ inline size_t gemm_tc_smem_bytes(int Ncp) {
    return (size_t)TC_STAGES * ((size_t)TC_BM * TC_BK * 4 + (size_t)Ncp * TC_BK * 4) + 1024 /*alignment*/ + 128 /*barriers, tmem address*/;
}

// shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled:
// 8-row groups 1024 bytes apart (stride offset), leading offset unused (1), descriptor version 1.
__device__ __forceinline__ unsigned long long tc_smem_desc(unsigned addr) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3FFF);
    d |= (unsigned long long)1 << 16;
    d |= (unsigned long long)(1024 >> 4) << 32;
    d |= (unsigned long long)1 << 46;
    d |= (unsigned long long)2 << 61;    // SWIZZLE_128B
    return d;
}
// instruction descriptor: D = F32, A = B = TF32, both K-major, N and M encoded as N/8 and M/16
__device__ __forceinline__ unsigned tc_idesc(int n) {
    return (1u << 4) | (2u << 7) | (2u << 10) | ((unsigned)(n >> 3) << 17) | ((unsigned)(TC_BM >> 4) << 24);
}
// 32 lanes x 8 consecutive columns of tensor memory -> 8 registers per thread (lane = row of the accumulator)
__device__ __forceinline__ void tmem_ld8(unsigned taddr, unsigned (&v)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_mma_tf32(unsigned d, unsigned long long da, unsigned long long db, unsigned idesc, unsigned acc) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tc_commit(unsigned bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tma_load_3d_sw(unsigned dst, const CUtensorMap* map, int x, int y, int z, unsigned bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];\n"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}

__global__ void __launch_bounds__(TC_THREADS, 1)
k_gemm_tf32(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmTcArgs a) {
    extern __shared__ __align__(16) unsigned char tc_smem_raw[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned a_bytes = TC_BM * TC_BK * 4, b_bytes = (unsigned)a.Ncp * TC_BK * 4;
    const unsigned stage_bytes = a_bytes + b_bytes;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(base + (size_t)TC_STAGES * stage_bytes);
    const unsigned bar_full = smem_u32(bars), bar_empty = bar_full + 8 * TC_STAGES, bar_acc = bar_empty + 8 * TC_STAGES;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 2 * TC_STAGES + 1);
    const unsigned smem_base = smem_u32(base);

    const int mt = blockIdx.x, sp = blockIdx.y, c = blockIdx.z;
    const int KB = (a.K + TC_BK - 1) / TC_BK;
    const int kb0 = sp * a.kb_per_split;
    const int nkb = max(0, min(KB, kb0 + a.kb_per_split) - kb0);
    unsigned ncols = 32;                       // tensor-memory columns: power of two >= Ncp
    while ((int)ncols < a.Ncp) ncols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        mbar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const unsigned tmem = *tmem_slot;
    bool dead = false;

    if (warp == 0) {
        // ---- TMA producer ----
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % TC_STAGES;
                if (kb >= TC_STAGES) mbar_wait_ready(bar_empty + 8 * s, (unsigned)((kb / TC_STAGES - 1) & 1), a.flags, dead);
                const unsigned dst = smem_base + s * stage_bytes;
                mbar_expect_tx(bar_full + 8 * s, stage_bytes);
                tma_load_3d_sw(dst, &tmA, (kb0 + kb) * TC_BK, mt * TC_BM, c, bar_full + 8 * s);
                tma_load_3d_sw(dst + a_bytes, &tmB, (kb0 + kb) * TC_BK, 0, c, bar_full + 8 * s);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        if (lane == 0) {
            const unsigned idesc = tc_idesc(a.Ncp);
            for (int kb = 0; kb < nkb; ++kb) {
                const int s = kb % TC_STAGES;
                mbar_wait_ready(bar_full + 8 * s, (unsigned)((kb / TC_STAGES) & 1), a.flags, dead);
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const unsigned long long da = tc_smem_desc(smem_base + s * stage_bytes);
                const unsigned long long db = tc_smem_desc(smem_base + s * stage_bytes + a_bytes);
#pragma unroll
                for (int k = 0; k < TC_BK / 8; ++k) {
                    const unsigned acc = (kb > 0 || k > 0) ? 1u : 0u;
                    // 8 floats of K = 32 bytes further along the swizzled row: start address field + 2
                    asm volatile(
                        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"
                        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}\n"
                        ::"r"(tmem), "l"(da + (unsigned long long)(2 * k)), "l"(db + (unsigned long long)(2 * k)), "r"(idesc), "r"(acc) : "memory");
                }
                // the stage may be refilled once these MMAs have read it
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar_empty + 8 * s) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar_acc) : "memory");
        }
    } else {
        // ---- epilogue: tensor memory -> registers -> Cpart ----
        mbar_wait(bar_acc, 0u, a.flags, dead);
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const int quarter = warp & 3;                    // the tensor-memory lanes this warp may read
        const int row = mt * TC_BM + quarter * 32 + lane;
        float* out = a.Cpart + (((size_t)c * a.S + sp) * a.M + row) * a.Ncp;
        for (int col = 0; col < a.Ncp; col += 8) {
            unsigned r[8];
            const unsigned taddr = tmem + ((unsigned)(quarter * 32) << 16) + (unsigned)col;
            if (nkb > 0) {
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                             : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                             : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) r[j] = 0u;
            }
            if (row < a.M) {
                *reinterpret_cast<uint4*>(out + col) = make_uint4(r[0], r[1], r[2], r[3]);
                *reinterpret_cast<uint4*>(out + col + 4) = make_uint4(r[4], r[5], r[6], r[7]);
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(ncols) : "memory");
    }
}

// C[c][row][col] = sum_s Cpart[c][s][row][col], col < Nc  (fixed order).  One thread per output.
__global__ void k_gemm_reduce(const float* Cpart, float* C, int M, int Nc, int Ncp, int S, int count) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    size_t per = (size_t)M * Nc;
    if (idx >= per * count) return;
    int c = (int)(idx / per);
    size_t e = idx % per;
    int row = (int)(e / Nc), col = (int)(e % Nc);
    float s = 0.f;
    for (int k = 0; k < S; ++k) s += Cpart[(((size_t)c * S + k) * M + row) * Ncp + col];
    C[idx] = s;
}

// Out[c][j][i] = In[c][i][j]  (rows x cols -> cols x rows), 32 x 32 tiles through shared memory.
__global__ void k_transpose(const float* In, float* Out, int rows, int cols) {
    __shared__ float t[32][33];
    const float* ib = In + (size_t)blockIdx.z * rows * cols;
    float* ob = Out + (size_t)blockIdx.z * rows * cols;
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        int r = r0 + j, cidx = c0 + threadIdx.x;
        t[j][threadIdx.x] = (r < rows && cidx < cols) ? ib[(size_t)r * cols + cidx] : 0.f;
    }
    __syncthreads();
    for (int j = threadIdx.y; j < 32; j += blockDim.y) {
        int cidx = c0 + j, r = r0 + threadIdx.x;
        if (cidx < cols && r < rows) ob[(size_t)cidx * rows + r] = t[threadIdx.x][j];
    }
}

}  // namespace psgd

namespace psgd {

// ---------------------------------------------------------------------------------------------
// Residual update on the tensor cores for ranks above 16:  E_i = M_i - P~ Q_i^T  (Algorithm 2, last
// line; with M == nullptr the dense reconstruction P~ Q^T of Algorithm 1).  The rank-r product is a
// 128 x 128 output tile with K = r, accumulated in tensor memory; float32 accuracy comes from
// splitting both small factors exactly into three TF32 numbers (x = h + m + l, 11 + 11 + 2 mantissa
// bits) and issuing the six products down to 2^-22 (l*h, h*l, m*m, m*h, h*m, h*h, small terms
// first), so that what is dropped (m*l, l*m, l*l) is below 2^-33 relative.  The epilogue
// warps read the accumulator back (tcgen05.ld), subtract it from M and store E.  Tensor memory
// holds two accumulators, so the MMAs of the next column tile overlap the epilogue of this one.
// ---------------------------------------------------------------------------------------------
constexpr int RT_BN = 128;        // columns per output tile (= UMMA N)
constexpr int RT_STAGES = 2;
constexpr int RT_XPOSE_BYTES = 32 * 32 * 4;   // per epilogue warp: one 32 x 32 block turned from row-per-lane to row-contiguous
constexpr int RT_THREADS = 320;   // warp 0: TMA, warp 1: MMA + tensor-memory owner, warps 2-9: epilogue (two per lane quarter)

struct ResidTcArgs {
    const float* M;     // [mats][rows][n] or nullptr
    float* Out;         // [mats][rows][n] (may alias M)
    int rows, n, KP;    // KP: rank padded to a multiple of 32
    int nodes;          // matrices per P~ (node count), 1 when Out is per matrix only
    int q_per_node;     // 1: Q indexed like Out (matrix, node); 0: by matrix only
    int* flags;
};

__host__ __device__ inline size_t resid_tc_smem_bytes() {
    return (size_t)RT_STAGES * (3 * TC_BM * TC_BK * 4 + 3 * RT_BN * TC_BK * 4) + 8 * RT_XPOSE_BYTES + 1024 + 256;
}

// X [rows][r] -> Xh, Xm, Xl [rows][KP], zero padded: x = h + m + l exactly, each term a TF32 number
// (h: x with its 13 low mantissa bits cleared; m: the same of x - h; l: what is left, at most 2 bits).
__global__ void k_split_pad(const float* X, float* Xh, float* Xm, float* Xl, size_t rows, int r, int KP) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * KP) return;
    size_t row = idx / KP;
    int k = (int)(idx % KP);
    float x = (k < r) ? X[row * r + k] : 0.f;
    float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    float r1 = x - h;
    float mm = __uint_as_float(__float_as_uint(r1) & 0xFFFFE000u);
    Xh[idx] = h;
    Xm[idx] = mm;
    Xl[idx] = r1 - mm;
}

__global__ void __launch_bounds__(RT_THREADS, 1)
k_residual_tc(const __grid_constant__ CUtensorMap tmPh, const __grid_constant__ CUtensorMap tmPm, const __grid_constant__ CUtensorMap tmPl,
              const __grid_constant__ CUtensorMap tmQh, const __grid_constant__ CUtensorMap tmQm, const __grid_constant__ CUtensorMap tmQl,
              ResidTcArgs a) {
    extern __shared__ __align__(16) unsigned char rt_smem_raw[];
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(rt_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr unsigned A_BYTES = TC_BM * TC_BK * 4, B_BYTES = RT_BN * TC_BK * 4;
    constexpr unsigned STAGE_BYTES = 3 * A_BYTES + 3 * B_BYTES;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(base + (size_t)RT_STAGES * STAGE_BYTES);
    const unsigned bar_full = smem_u32(bars), bar_empty = bar_full + 8 * RT_STAGES;
    const unsigned bar_accf = bar_empty + 8 * RT_STAGES, bar_acce = bar_accf + 16;   // accumulator full / free, 2 each
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 2 * RT_STAGES + 4);
    const unsigned smem_base = smem_u32(base);

    const int rt = blockIdx.x, mat = blockIdx.y;
    const int c = mat / a.nodes;                    // matrix index of P~
    const int qz = a.q_per_node ? mat : c;          // which Q
    const int nct = (a.n + RT_BN - 1) / RT_BN;      // column tiles
    const int nkc = a.KP / TC_BK;                   // K chunks per tile
    const int total = nct * nkc;

    if (tid == 0) {
        for (int s = 0; s < RT_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(bar_accf + 8 * b, 1); mbar_init(bar_acce + 8 * b, 8); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(4u * RT_BN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const unsigned tmem = *tmem_slot;
    bool dead = false;

    if (warp == 0) {
        // ---- TMA producer: per (column tile, K chunk) the heads and tails of both factors ----
        if (lane == 0) {
            for (int it = 0, ct = 0, kc = 0; it < total; ++it, ct += (kc + 1 == nkc), kc = (kc + 1 == nkc) ? 0 : kc + 1) {
                const int s = it % RT_STAGES;
                if (it >= RT_STAGES) mbar_wait_ready(bar_empty + 8 * s, (unsigned)((it / RT_STAGES - 1) & 1), a.flags, dead);
                const unsigned dst = smem_base + s * STAGE_BYTES;
                const unsigned bar = bar_full + 8 * s;
                mbar_expect_tx(bar, STAGE_BYTES);
                const int kx = (nkc - 1 - kc) * TC_BK;      // last columns of the factors first (see the MMA issuer)
                tma_load_3d_sw(dst, &tmPh, kx, rt * TC_BM, c, bar);
                tma_load_3d_sw(dst + A_BYTES, &tmPm, kx, rt * TC_BM, c, bar);
                tma_load_3d_sw(dst + 2 * A_BYTES, &tmPl, kx, rt * TC_BM, c, bar);
                tma_load_3d_sw(dst + 3 * A_BYTES, &tmQh, kx, ct * RT_BN, qz, bar);
                tma_load_3d_sw(dst + 3 * A_BYTES + B_BYTES, &tmQm, kx, ct * RT_BN, qz, bar);
                tma_load_3d_sw(dst + 3 * A_BYTES + 2 * B_BYTES, &tmQl, kx, ct * RT_BN, qz, bar);
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer ----
        if (lane == 0) {
            const unsigned idesc = tc_idesc(RT_BN);
            for (int it = 0, ct = 0, kc = 0; it < total; ++it, ct += (kc + 1 == nkc), kc = (kc + 1 == nkc) ? 0 : kc + 1) {
                const int s = it % RT_STAGES;
                const int ab = ct & 1;                                   // accumulator buffer
                if (kc == 0 && ct >= 2) mbar_wait_ready(bar_acce + 8 * ab, (unsigned)(((ct >> 1) - 1) & 1), a.flags, dead);
                mbar_wait_ready(bar_full + 8 * s, (unsigned)((it / RT_STAGES) & 1), a.flags, dead);
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const unsigned sb = smem_base + s * STAGE_BYTES;
                const unsigned long long dP[3] = {tc_smem_desc(sb), tc_smem_desc(sb + A_BYTES), tc_smem_desc(sb + 2 * A_BYTES)};
                const unsigned long long dQ[3] = {tc_smem_desc(sb + 3 * A_BYTES), tc_smem_desc(sb + 3 * A_BYTES + B_BYTES),
                                                  tc_smem_desc(sb + 3 * A_BYTES + 2 * B_BYTES)};
                // two accumulators per tile: the h*h products (8 adds per 64 of K) and the five small products,
                // so that the rounding of the tensor core's float32 adds hits the large running sum as rarely as possible.
                // That add truncates toward zero, about 3e-8 of the running sum each time; the columns of P~ Q_i^T are
                // summed from the last to the first because the leading columns carry the large terms (P~ comes out of
                // a QR of M Q, or of Ritz vectors sorted by singular value): the running sum stays small until the end.
                const unsigned d_big = tmem + (unsigned)(ab * 2 * RT_BN), d_small = d_big + RT_BN;
                // (index of the P term, index of the Q term) with h = 0, m = 1, l = 2; small products first
                const int tp[6] = {2, 0, 1, 1, 0, 0}, tq[6] = {0, 2, 1, 0, 1, 0};
#pragma unroll
                for (int k = 0; k < TC_BK / 8; ++k) {
                    const unsigned long long o = (unsigned long long)(2 * (TC_BK / 8 - 1 - k));
#pragma unroll
                    for (int t = 0; t < 6; ++t) {
                        const unsigned acc = (kc > 0 || k > 0 || (t > 0 && t < 5)) ? 1u : 0u;
                        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}\n"
                                     ::"r"(t == 5 ? d_big : d_small), "l"(dP[tp[t]] + o), "l"(dQ[tq[t]] + o), "r"(idesc), "r"(acc) : "memory");
                    }
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar_empty + 8 * s) : "memory");
                if (kc == nkc - 1)
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar_accf + 8 * ab) : "memory");
            }
        }
    } else {
        // ---- epilogue: E = M - accumulator ----
        // Eight warps: warp w reads the tensor-memory lanes of quarter w % 4 (its 32 accumulator rows) and the
        // 32-column chunks of parity (w - 2) / 4.  Tensor memory hands a thread one row of the block; written like
        // that to HBM every instruction would touch 32 lines, and the load-store unit, not HBM, would set the pace.
        // So the block goes through a 4 KB shared-memory buffer of the warp (16-byte units XOR-swizzled by row) and
        // comes back as 4 rows x 128 contiguous bytes per instruction, the layout M is loaded and E stored in.
        // The M values of the next chunk are requested before the accumulator is read.
        const int quarter = warp & 3;
        const int half = (warp - 2) >> 2;
        float4* xb = reinterpret_cast<float4*>(base + (size_t)RT_STAGES * STAGE_BYTES + 256 + (size_t)(warp - 2) * RT_XPOSE_BYTES);
        const int lrow = lane >> 3, lch = lane & 7;           // coalesced phase: row within a group of 4, 16-byte unit
        const int brow0 = rt * TC_BM + quarter * 32;          // first row of this warp's blocks
        const size_t mrow = (size_t)mat * a.rows;
        auto load_m = [&](int col0, float4 (&dst)[8]) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int row = brow0 + 4 * i + lrow, col = col0 + 4 * lch;
                dst[i] = (a.M && row < a.rows && col < a.n) ? ldg_stream4(a.M + (mrow + row) * a.n + col) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        };
        float4 mv[8];
        load_m(half * 32, mv);
        for (int ct = 0; ct < nct; ++ct) {
            const int ab = ct & 1;
            mbar_wait(bar_accf + 8 * ab, (unsigned)((ct >> 1) & 1), a.flags, dead);
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
#pragma unroll 1
            for (int cc = half * 32; cc < RT_BN; cc += 64) {
                const int col0 = ct * RT_BN + cc;
                // next chunk of this warp: the other chunk of this tile, else the first chunk of the next tile
                const int cnext = (cc + 64 < RT_BN) ? col0 + 64 : (ct + 1) * RT_BN + half * 32;
                float4 mn[8];
                load_m(cnext < a.n && (cc + 64 < RT_BN || ct + 1 < nct) ? cnext : a.n, mn);
                if (col0 < a.n) {
                    const unsigned taddr = tmem + ((unsigned)(quarter * 32) << 16) + (unsigned)(ab * 2 * RT_BN + cc);
#pragma unroll
                    for (int p8 = 0; p8 < 4; ++p8) {
                        unsigned rb[8], rs[8];
                        tmem_ld8(taddr + 8 * p8, rb);
                        tmem_ld8(taddr + (unsigned)RT_BN + 8 * p8, rs);
                        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int j = 2 * p8 + q;            // 16-byte unit of this lane's row
                            xb[lane * 8 + (j ^ (lane & 7))] =
                                make_float4(__uint_as_float(rb[4 * q]) + __uint_as_float(rs[4 * q]),
                                            __uint_as_float(rb[4 * q + 1]) + __uint_as_float(rs[4 * q + 1]),
                                            __uint_as_float(rb[4 * q + 2]) + __uint_as_float(rs[4 * q + 2]),
                                            __uint_as_float(rb[4 * q + 3]) + __uint_as_float(rs[4 * q + 3]));
                        }
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int br = 4 * i + lrow, row = brow0 + br, col = col0 + 4 * lch;
                        const float4 pq = xb[br * 8 + (lch ^ (br & 7))];
                        if (row < a.rows && col < a.n) {       // n % 4 == 0: a group of 4 columns is all in or all out
                            float4 o;
                            if (a.M) o = make_float4(mv[i].x - pq.x, mv[i].y - pq.y, mv[i].z - pq.z, mv[i].w - pq.w);
                            else o = pq;
                            *reinterpret_cast<float4*>(a.Out + (mrow + row) * a.n + col) = o;
                        }
                    }
                    __syncwarp();
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) mv[i] = mn[i];
            }
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acce + 8 * ab);      // this warp is done with the accumulator buffer
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(4u * RT_BN) : "memory");
    }
}

}  // namespace psgd

namespace psgd {

// ---------------------------------------------------------------------------------------------
// Projection on the tensor cores (ranks above 16; with the pending residual of the two-pass deferred mode
// from 9 columns on):  P_i = (A_i [+ B_i]) Q  (Algorithm 1: P^(i) <- Delta^(i) Q, with the error-feedback
// add of Eq. (7a) fused in; optionally stores M = A + B).
// Per 32-column K block TMA brings the 128 x 32 tiles of A and B (128-byte swizzled); eight
// converter warps form M in place of A and write it back to HBM.  M is used as two TF32 terms: the
// head is M itself (the tensor core reads a float32 as TF32, i.e. truncated), the second term is
// M - head rounded to the nearest TF32 number, written over the tile of B; what is left (at most
// 2^-21 |M|, zero mean) averages out over the hundreds of columns of a sum.  Q^T arrives pre-split
// into three exact terms, one untiled bulk copy per K block of an image in shared-memory order
// (k_split_img_t).  Products: h x [h|m|l] and m x [h|m]; m x l is below 2^-32.
//
// Accumulation.  The tensor core adds to its float32 accumulator with truncation (measured on
// like-signed sums: 3e-8 relative per accumulation, always toward zero, i.e. 2e-5 over the 512
// steps of a 4096-long contraction).  The head product therefore accumulates one K block (4 steps)
// at a time in tensor memory: accumulators take turns, and eight adder warps add each finished one
// to float32 registers (round to nearest) while the next ones fill.  Adding up after every 2 steps
// halves the bias again but was 25 % slower: every hand-over lengthens the life of a pipeline stage.
//   up to 80 columns: the three terms of Q^T lie side by side as one B operand of 3 Ncp <= 256 rows:
//     two MMAs per 8 of K into an accumulator set [head | small | small], all of it added up per K block;
//   above: three MMAs (h x h, h x [m|l], m x [h|m]); the small products keep two accumulators for the
//     whole contraction, the head product goes through the rotating accumulators.
// One mbarrier per K block ("done", by tcgen05.commit) frees the shared-memory stages and tells the
// adder warps that the accumulators of that K block can be read.
// ---------------------------------------------------------------------------------------------
constexpr int PT_THREADS = 576;   // warp 0: TMA, warp 1: MMA + tensor-memory owner, warps 2-9: converters, warps 10-17: adders + epilogue
constexpr int PT_THREADS_PEND = 608;   // ... and warp 18: issues the MMAs of the pending-residual correction
constexpr int BT_MAXG = 8;        // 8-column groups per thread: (Ncp / 2) / 8 for Ncp <= 128

// Adder warps of the projection and back-projection kernels: adds the accumulators of one K block (set / head
// accumulator hb) to the thread's float32 registers.  The thread owns tensor-memory lane (lane_base) and the ng groups
// of 8 columns starting at col_base.  wide: the set is [head | small | small] at 3 hb Ncp; else the head accumulator
// at (2 + hb) Ncp (the two small accumulators at 0 stay for the whole contraction).
__device__ __forceinline__ void tc_add_up(float (&acc)[BT_MAXG][8], unsigned tmem, unsigned lane_base, unsigned col_base,
                                          int Ncp, int ng, bool wide, int hb) {
    if (wide) {
        const unsigned ts = tmem + lane_base + (unsigned)(3 * hb * Ncp) + col_base;
#pragma unroll
        for (int g = 0; g < 5; ++g) {              // Ncp <= 80: at most 5 groups of 8 columns per thread
            if (g < ng) {
                unsigned vh[8], v1[8], v2[8];
                tmem_ld8(ts + 8 * g, vh);
                tmem_ld8(ts + (unsigned)Ncp + 8 * g, v1);
                tmem_ld8(ts + (unsigned)(2 * Ncp) + 8 * g, v2);
                asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[g][j] += __uint_as_float(vh[j]) + (__uint_as_float(v1[j]) + __uint_as_float(v2[j]));
            }
        }
    } else {
        const unsigned t0 = tmem + lane_base + (unsigned)((2 + hb) * Ncp) + col_base;
#pragma unroll
        for (int g2 = 0; g2 < BT_MAXG; g2 += 2) {
            if (g2 < ng) {
                unsigned v0[8], v1[8];
                tmem_ld8(t0 + 8 * g2, v0);
                if (g2 + 1 < ng) tmem_ld8(t0 + 8 * (g2 + 1), v1);
                asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[g2][j] += __uint_as_float(v0[j]);
                if (g2 + 1 < ng) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) acc[g2 + 1][j] += __uint_as_float(v1[j]);
                }
            }
        }
    }
}
// The small accumulators (not wide) added to the registers of column group g; wide: nothing is left in tensor memory.
__device__ __forceinline__ void tc_add_small(float (&v)[8], const float (&acc)[8], unsigned tmem, unsigned lane_base, unsigned col_base,
                                             int Ncp, bool wide, int g) {
    if (!wide) {
        unsigned s1[8], s2[8];
        tmem_ld8(tmem + lane_base + col_base + 8 * g, s1);
        tmem_ld8(tmem + lane_base + (unsigned)Ncp + col_base + 8 * g, s2);
        asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = acc[j] + (__uint_as_float(s1[j]) + __uint_as_float(s2[j]));
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = acc[j];
    }
}

struct ProjTcArgs {
    float* Mout;      // [mats][rows][n] or nullptr
    float* P;         // [mats][rows][r]
    int rows, n, r, Ncp, nh, has_b;
    int nodes;        // matrices per Q
    int* flags;
    const int* skip;
    // pending residual (two-pass deferred mode): M = A + (B - P~_prev Qsub^T), the product formed by the tensor core
    const float* Pimg;    // [count][row tiles][2][128][32]: two TF32 terms of P~_prev, shared-memory image (k_split_img_rows)
    const float* QSimg;   // [mats or count][groups][3][32][32]: three terms of Qsub, one image per group of K blocks (k_split_img_qs)
    int qs_per_node;      // Qsub is per (matrix, node) (1) or per matrix (0)
    int ksteps;           // ceil(r / 8): MMAs along the rank
    int qs_group;         // K blocks per image: 4 (r <= 8), 2 (r <= 16) or 1; their 32 / qs_group rank columns lie side by side in a row
    int qs_groups;        // images per matrix: ceil(KB / qs_group)
};
constexpr int PT_NQ = 3;                             // stages of the ring of Qsub images (pend)
constexpr int PT_CORR_COLS = 96;                     // one correction accumulator: [head | small | small] x 32 columns
constexpr unsigned PT_QS_BYTES = 3 * 32 * TC_BK * 4; // three terms of a 32-row block of Qsub
constexpr unsigned PT_PIMG_BYTES = 2 * TC_BM * TC_BK * 4;

// Two shared-memory rings, as in the back-projection below: stages of 32 KB for the tiles of A and B (M and its second
// TF32 term are formed in place) and a short ring for the three terms of Q^T.
// (pend: the two terms of P~_prev stay resident, and the images of Qsub have a ring of their own, filled by the thread that
// issues the correction MMAs and released as soon as those have completed, so that it runs ahead of the other rings)
__host__ __device__ inline int proj_tc_nm(int Ncp) { return 3 * Ncp <= 256 ? 3 : 2; }
__host__ __device__ inline long long proj_tc_short_bytes(int Ncp) { return 3ll * Ncp * TC_BK * 4; }
__host__ __device__ inline long long proj_tc_pend_bytes(bool pend) { return pend ? (long long)PT_PIMG_BYTES + (long long)PT_NQ * PT_QS_BYTES : 0; }
__host__ __device__ inline int proj_tc_nh(int Ncp, bool pend = false) {
    const long long left = 224ll * 1024 - 1024 - 512 - proj_tc_nm(Ncp) * proj_tc_short_bytes(Ncp) - proj_tc_pend_bytes(pend);
    const int nh = (int)(left / (2 * TC_BM * TC_BK * 4));
    return nh > 6 ? 6 : nh;
}
__host__ __device__ inline size_t proj_tc_smem_bytes(int Ncp, bool pend = false) {
    return (size_t)proj_tc_nh(Ncp, pend) * 2 * TC_BM * TC_BK * 4 + (size_t)(proj_tc_nm(Ncp) * proj_tc_short_bytes(Ncp)) +
           (size_t)proj_tc_pend_bytes(pend) + 1024 + 512;
}

// Q [count][n][r] -> Qimg[count][KB][t][Ncp][32], t = 0, 1, 2: the transposed factor split exactly into three TF32 terms
// (h = x with its 13 low mantissa bits cleared, m the same of x - h, l the rest), laid out as the shared-memory
// image of one K block after the other (rows of 128 bytes, 128-byte swizzle: the 16-byte unit u of row k sits at unit
// u ^ (k & 7)), so that ONE untiled bulk copy of 3 Ncp 128 bytes brings what a K block needs.  Columns beyond n and rows
// k >= r are zero.  One thread per (matrix, K block, k, column).
__global__ void k_split_img_t(const float* Q, float* Qimg, int n, int r, int Ncp, int KB, int count, const int* skip) {
    if (skip && *skip) return;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t per_kb = (size_t)Ncp * TC_BK, tot = per_kb * KB * count;
    if (idx >= tot) return;
    const int c = (int)(idx / (per_kb * KB));
    const int kb = (int)((idx / per_kb) % KB);
    const int k = (int)((idx % per_kb) / TC_BK), cc = (int)(idx % TC_BK);
    const int col = kb * TC_BK + cc;
    float x = (k < r && col < n) ? Q[((size_t)c * n + col) * r + k] : 0.f;
    float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    float r1 = x - h;
    float mm = __uint_as_float(__float_as_uint(r1) & 0xFFFFE000u);
    float* blk = Qimg + ((size_t)c * KB + kb) * 3 * per_kb;
    const size_t o = (size_t)k * TC_BK + ((((cc >> 2) ^ (k & 7)) << 2) | (cc & 3));
    blk[o] = h;
    blk[per_kb + o] = mm;
    blk[2 * per_kb + o] = r1 - mm;
}
// X [mats][rows][r] -> img[mats][ceil(rows / TR)][T][TR][32]: blocks of TR rows as K-major shared-memory images (rows of 128
// bytes holding columns 0..31, zero beyond r and beyond `rows`; 128-byte swizzle).  T = 3: the three exact TF32 terms;
// T = 2: head and the rest rounded to the nearest TF32 number.  One thread per (matrix, row, column).
__global__ void k_split_img_rows(const float* X, float* img, int rows, int r, int TR, int T, int mats) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int tiles = (rows + TR - 1) / TR;
    const size_t per_mat = (size_t)tiles * TR * TC_BK, tot = per_mat * mats;
    if (idx >= tot) return;
    const int mt = (int)(idx / per_mat);
    const size_t w = idx % per_mat;
    const int tile = (int)(w / ((size_t)TR * TC_BK)), rr = (int)((w / TC_BK) % TR), k = (int)(w % TC_BK);
    const int row = tile * TR + rr;
    const float x = (row < rows && k < r) ? X[((size_t)mt * rows + row) * r + k] : 0.f;
    const float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    const float r1 = x - h;
    float* blk = img + ((size_t)mt * tiles + tile) * T * TR * TC_BK;
    const size_t o = (size_t)rr * TC_BK + ((((k >> 2) ^ (rr & 7)) << 2) | (k & 3));
    blk[o] = h;
    if (T == 2) {
        blk[(size_t)TR * TC_BK + o] = __uint_as_float((__float_as_uint(r1) + 0x1000u) & 0xFFFFE000u);
    } else {
        const float mm = __uint_as_float(__float_as_uint(r1) & 0xFFFFE000u);
        blk[(size_t)TR * TC_BK + o] = mm;
        blk[2 * (size_t)TR * TC_BK + o] = r1 - mm;
    }
}
// Qsub [mats][n][r] -> img[mats][groups][3][32][32]: image gi holds the K blocks G gi .. G gi + G - 1 (32 rows of Qsub each).
// Row `row` of the image is [block 0: k = 0 .. 32/G - 1 | block 1 | ...] of those blocks' row `row`, as three exact TF32 terms,
// 128-byte swizzled; zero beyond r and beyond n.  One thread per (matrix, image, row, float).
__global__ void k_split_img_qs(const float* X, float* img, int n, int r, int G, int groups, int mats) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t per_img = 32 * TC_BK, tot = per_img * groups * mats;
    if (idx >= tot) return;
    const int mt = (int)(idx / (per_img * groups));
    const int gi = (int)((idx / per_img) % groups), row = (int)((idx / TC_BK) % 32), f = (int)(idx % TC_BK);
    const int kpad = TC_BK / G, q = f / kpad, k = f % kpad;
    const int col = (gi * G + q) * 32 + row;
    const float x = (col < n && k < r) ? X[((size_t)mt * n + col) * r + k] : 0.f;
    const float h = __uint_as_float(__float_as_uint(x) & 0xFFFFE000u);
    const float r1 = x - h;
    const float mm = __uint_as_float(__float_as_uint(r1) & 0xFFFFE000u);
    float* blk = img + ((size_t)mt * groups + gi) * 3 * per_img;
    const size_t o = (size_t)row * TC_BK + ((((f >> 2) ^ (row & 7)) << 2) | (f & 3));
    blk[o] = h;
    blk[per_img + o] = mm;
    blk[2 * per_img + o] = r1 - mm;
}
__device__ __forceinline__ void tmem_ld16(unsigned taddr, unsigned (&v)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void bulk_load_1d(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// PEND (two-pass deferred mode, up to 32 columns): the tile of B holds Delta_{t-1} and M = A + (B - P~_prev Qsub^T).  The
// rank-r product of a K block, C = P~_prev[128 rows] Qsub[32 columns]^T, is formed by the tensor core into one of two
// correction accumulators before the converters need it (P~_prev as two TF32 terms resident in shared memory, the block of
// Qsub as three terms in the short ring: h x [h|m|l] and m x [h|m], `ksteps` pairs of MMAs).  The converters then work one
// accumulator row per lane: they read C with tcgen05.ld, form M in the (swizzled, hence conflict-free) tile and its second
// term, and after a barrier among themselves write the tile of M back to HBM with the row-contiguous mapping.
#ifdef PSGD_PTC_TIMING
// Per-K-block time stamps of CTA (0, 0) (instrumented builds only): [event][K block], SM clock, low 32 bits.
__device__ unsigned g_ptc_t[12][512];
#define PTC_STAMP(ev, kb) do { if (blockIdx.x == 0 && blockIdx.y == 0 && (kb) < 512) g_ptc_t[ev][kb] = (unsigned)clock64(); } while (0)
#else
#define PTC_STAMP(ev, kb) do { } while (0)
#endif

template <bool PEND>
__global__ void __launch_bounds__(PEND ? PT_THREADS_PEND : PT_THREADS, 1)
k_project_tc(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const float* __restrict__ Qimg,
             ProjTcArgs a) {
    extern __shared__ __align__(16) unsigned char pt_smem_raw[];
    if (a.skip && *a.skip) return;
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(pt_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr unsigned A_BYTES = TC_BM * TC_BK * 4;
    constexpr unsigned LONG_BYTES = 2 * A_BYTES;               // [A tile -> M (head)][B tile -> second term]
    const unsigned B_BYTES = (unsigned)a.Ncp * TC_BK * 4;
    const unsigned SHORT_BYTES = 3 * B_BYTES;                  // h, m, l of Q^T
    const bool wide = 3 * a.Ncp <= 256;
    const int NM = proj_tc_nm(a.Ncp);
    const int CORR = PEND ? 2 * PT_CORR_COLS : 0;              // tensor-memory columns of the two correction accumulators
    const int NH = a.nh, NB = wide ? min(4, (512 - CORR) / (3 * a.Ncp)) : min(3, (512 - 2 * a.Ncp) / a.Ncp);
    unsigned char* short_base = base + (size_t)NH * LONG_BYTES;
    unsigned char* pimg_base = short_base + (size_t)NM * SHORT_BYTES;
    unsigned char* qs_base = pimg_base + (PEND ? PT_PIMG_BYTES : 0u);       // ring of Qsub images (pend)
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(qs_base + (PEND ? PT_NQ * PT_QS_BYTES : 0u));
    const unsigned bar_hfull = smem_u32(bars), bar_conv = bar_hfull + 8 * NH, bar_done = bar_conv + 8 * NH;
    const unsigned bar_bfull = bar_done + 8 * NH, bar_free = bar_bfull + 8 * NM, bar_acc = bar_free + 8 * NB;
    const unsigned bar_stored = bar_acc + 8, bar_corr = bar_stored + 8 * NH, bar_cfree = bar_corr + 16, bar_pfull = bar_cfree + 16;
    const unsigned bar_qfull = bar_pfull + 8, bar_qfree = bar_qfull + 8 * PT_NQ;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 4 * NH + NM + NB + 1 + 5 + 2 * PT_NQ);
    const unsigned ring_u32 = smem_u32(base), short_u32 = smem_u32(short_base), pimg_u32 = smem_u32(pimg_base), qs_u32 = smem_u32(qs_base);

    const int rt = blockIdx.x, mat = blockIdx.y;
    const int qz = mat / a.nodes;
    // the K blocks (32 columns each) of this row block are dealt to gridDim.z CTAs; with more than one the partial
    // products are added into a zeroed P (two addends per element: the sum does not depend on their order)
    const int KBt = (a.n + TC_BK - 1) / TC_BK;
    const int kb_lo = (int)((long long)KBt * blockIdx.z / gridDim.z);
    const int KB = (int)((long long)KBt * (blockIdx.z + 1) / gridDim.z) - kb_lo;
    unsigned ncols = 32;
    while ((int)ncols < CORR + (wide ? NB * 3 : NB + 2) * a.Ncp) ncols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < NH; ++s) {
            mbar_init(bar_hfull + 8 * s, 1); mbar_init(bar_conv + 8 * s, 4); mbar_init(bar_done + 8 * s, 1); mbar_init(bar_stored + 8 * s, 4);
        }
        for (int s = 0; s < NM; ++s) mbar_init(bar_bfull + 8 * s, 1);
        for (int b = 0; b < NB; ++b) mbar_init(bar_free + 8 * b, 8);
        mbar_init(bar_acc, 1);
        for (int b = 0; b < 2; ++b) { mbar_init(bar_corr + 8 * b, 1); mbar_init(bar_cfree + 8 * b, 4); }
        mbar_init(bar_pfull, 1);
        for (int b = 0; b < PT_NQ; ++b) { mbar_init(bar_qfull + 8 * b, 1); mbar_init(bar_qfree + 8 * b, 1); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const unsigned tmem_all = *tmem_slot;  // pend: correction accumulators at 0 and 96, the rest behind them
    const unsigned tmem = tmem_all + (unsigned)CORR;   // wide: set b at 3 b Ncp; else two small accumulators at 0, head b at (2 + b) Ncp
    bool dead = false;
    // K block j is "done" (all its MMAs have completed) in phase j / NH of bar_done[j % NH]
    auto wait_done = [&](int j) { mbar_wait(bar_done + 8 * (j % NH), (unsigned)((j / NH) & 1), a.flags, dead); };

    if (warp == 0) {
        // ---- TMA producer: tiles of A and B run NH - NM K blocks ahead of the terms of Q^T ----
        if (lane == 0) {
            const int lead = NH - NM;
            if (PEND) {
                mbar_expect_tx(bar_pfull, PT_PIMG_BYTES);
                bulk_load_1d(pimg_u32, a.Pimg + ((size_t)qz * gridDim.x + rt) * (PT_PIMG_BYTES / 4), PT_PIMG_BYTES, bar_pfull);
            }
            // (one thread: positions and parities as counters, a non-blocking test before every wait)
            int aj = 0, as = 0, aph = 1;             // next tile pair: index, stage j % NH, parity of "done"/"stored" of tile j - NH
            auto issue_ab = [&]() {
                if (aj >= NH) {
                    mbar_wait_ready(bar_done + 8 * as, (unsigned)aph, a.flags, dead);
                    if (PEND) mbar_wait_ready(bar_stored + 8 * as, (unsigned)aph, a.flags, dead);   // its M has left for HBM
                }
                const unsigned dst = ring_u32 + as * LONG_BYTES, bar = bar_hfull + 8 * as;
                PTC_STAMP(0, aj);
                mbar_expect_tx(bar, (a.has_b ? 2u : 1u) * A_BYTES);
                tma_load_3d_sw(dst, &tmA, (kb_lo + aj) * TC_BK, rt * TC_BM, mat, bar);
                if (a.has_b) tma_load_3d_sw(dst + A_BYTES, &tmB, (kb_lo + aj) * TC_BK, rt * TC_BM, mat, bar);
                ++aj;
                if (++as == NH) { as = 0; aph ^= 1; }
            };
            for (int j = 0; j < min(lead, KB); ++j) issue_ab();
            const float* qsrc = Qimg + ((size_t)qz * KBt + kb_lo) * (3u * B_BYTES / 4);
            int ss = 0, ds = 0, dph = 0;             // stage kb % NM; stage and parity of "done" of K block kb - NM
            for (int kb = 0; kb < KB; ++kb) {
                if (aj < KB) issue_ab();
                if (kb >= NM) {
                    mbar_wait_ready(bar_done + 8 * ds, (unsigned)dph, a.flags, dead);
                    if (++ds == NH) { ds = 0; dph ^= 1; }
                }
                const unsigned dst = short_u32 + ss * SHORT_BYTES, bar = bar_bfull + 8 * ss;
                mbar_expect_tx(bar, SHORT_BYTES);
                bulk_load_1d(dst, qsrc + (size_t)kb * (3u * B_BYTES / 4), 3u * B_BYTES, bar);
                if (++ss == NM) ss = 0;
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer: one thread, so every instruction of its loop is on the critical path of the whole CTA.  Ring
        //      positions and barrier parities are carried along as counters (no division), descriptors are offsets from
        //      those of stage 0 (the address field holds addr >> 4 and shared memory ends below 2^18). ----
        if (lane == 0) {
            const unsigned id1 = tc_idesc(a.Ncp), id2 = tc_idesc(2 * a.Ncp), id3 = tc_idesc(wide ? 3 * a.Ncp : a.Ncp);
            const unsigned long long dA0 = tc_smem_desc(ring_u32), dS0 = tc_smem_desc(short_u32);
            const unsigned long long long_step = LONG_BYTES >> 4, short_step = SHORT_BYTES >> 4;
            const unsigned long long a_off = A_BYTES >> 4, b_off = B_BYTES >> 4;
            int sh = 0, phh = 0, sm = 0, phm = 0, hb = 0, phb = 1;     // kb % NH, (kb / NH) & 1, ... ; phb: parity of kb / NB - 1
            for (int kb = 0; kb < KB; ++kb) {
                PTC_STAMP(10, kb);
                mbar_wait_ready(bar_conv + 8 * sh, (unsigned)phh, a.flags, dead);
                PTC_STAMP(11, kb);
                mbar_wait_ready(bar_bfull + 8 * sm, (unsigned)phm, a.flags, dead);
                if (kb >= NB) mbar_wait_ready(bar_free + 8 * hb, (unsigned)phb, a.flags, dead);   // registers took its last content
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                PTC_STAMP(5, kb);
                const unsigned long long dAh = dA0 + (unsigned long long)sh * long_step, dAm = dAh + a_off;
                const unsigned long long dQh = dS0 + (unsigned long long)sm * short_step, dQm = dQh + b_off;
                if (wide) {
                    const unsigned d_set = tmem + (unsigned)(3 * hb * a.Ncp);
#pragma unroll
                    for (int k = 0; k < TC_BK / 8; ++k) {
                        const unsigned long long o = (unsigned long long)(2 * k);
                        tc_mma_tf32(d_set, dAh + o, dQh + o, id3, k > 0 ? 1u : 0u);                        // h x [h|m|l]
                        tc_mma_tf32(d_set + (unsigned)a.Ncp, dAm + o, dQh + o, id2, 1u);                   // m x [h|m]
                    }
                } else {
                    const unsigned d_small = tmem, d_head = tmem + (unsigned)((2 + hb) * a.Ncp);
#pragma unroll
                    for (int k = 0; k < TC_BK / 8; ++k) {
                        const unsigned long long o = (unsigned long long)(2 * k);
                        tc_mma_tf32(d_small, dAh + o, dQm + o, id2, (kb > 0 || k > 0) ? 1u : 0u);          // h x [m|l]
                        tc_mma_tf32(d_small, dAm + o, dQh + o, id2, 1u);                                   // m x [h|m]
                        tc_mma_tf32(d_head, dAh + o, dQh + o, id1, k > 0 ? 1u : 0u);                       // h x h
                    }
                }
                PTC_STAMP(8, kb);
                tc_commit(bar_done + 8 * sh);
                PTC_STAMP(9, kb);
                if (++sh == NH) { sh = 0; phh ^= 1; }
                if (++sm == NM) { sm = 0; phm ^= 1; }
                if (++hb == NB) { hb = 0; phb ^= 1; }
            }
            tc_commit(bar_acc);
        }
    } else if (warp < 10) {
        // ---- converters: two groups of four warps (one warp per quarter of the tensor-memory lanes) take the K blocks in
        //      turn, so that the waits of one K block (tile arrival, tensor-memory reads, the group's barrier, the stores)
        //      overlap the arithmetic of the next ----
        const int grp = (warp - 2) >> 2;
        const int ct = tid - 64 - 128 * grp;           // 0 .. 127 within the group
        if (PEND) {
            // one accumulator row per lane: M = A + B - C, second term, then the tile of M to HBM
            const int quarter = warp & 3;              // tensor-memory lanes of this warp
            const int row = quarter * 32 + lane;
            const unsigned lane_base = (unsigned)(quarter * 32) << 16;
            for (int kb = grp; kb < KB; kb += 2) {
                const int sh = kb % NH, cb = grp;      // correction accumulator kb & 1
                mbar_wait_warp(bar_hfull + 8 * sh, (unsigned)((kb / NH) & 1), a.flags, dead);
                if (quarter == 2 && lane == 0) PTC_STAMP(1, kb);
                mbar_wait_warp(bar_corr + 8 * cb, (unsigned)((kb >> 1) & 1), a.flags, dead);
                if (quarter == 2 && lane == 0) PTC_STAMP(2, kb);
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                float4* t0 = reinterpret_cast<float4*>(base + (size_t)sh * LONG_BYTES);
                float4* t1 = t0 + A_BYTES / 16;
#pragma unroll
                for (int chalf = 0; chalf < 2; ++chalf) {
                    unsigned ch[16], c1[16], c2[16];
                    const unsigned tc = tmem_all + lane_base + (unsigned)(cb * PT_CORR_COLS + 16 * chalf);
                    tmem_ld16(tc, ch);
                    tmem_ld16(tc + 32u, c1);
                    tmem_ld16(tc + 64u, c2);
                    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
                    if (chalf == 1) {
                        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_cfree + 8 * cb);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int o = row * 8 + ((4 * chalf + j) ^ (row & 7));       // 16-byte unit of the swizzled tile
                        const float4 g = t0[o], e = t1[o];
                        float xs[4] = {g.x + e.x, g.y + e.y, g.z + e.z, g.w + e.w};
                        float ms[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            xs[q] -= __uint_as_float(ch[4 * j + q]) + (__uint_as_float(c1[4 * j + q]) + __uint_as_float(c2[4 * j + q]));
                            const float h = __uint_as_float(__float_as_uint(xs[q]) & 0xFFFFE000u);
                            ms[q] = __uint_as_float((__float_as_uint(xs[q] - h) + 0x1000u) & 0xFFFFE000u);
                        }
                        t0[o] = make_float4(xs[0], xs[1], xs[2], xs[3]);
                        t1[o] = make_float4(ms[0], ms[1], ms[2], ms[3]);
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");    // generic writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_conv + 8 * sh);
                if (quarter == 2 && lane == 0) PTC_STAMP(3, kb);
                if (grp == 0) asm volatile("bar.sync 1, 128;\n" ::: "memory");    // every row of M is in the tile
                else asm volatile("bar.sync 2, 128;\n" ::: "memory");
#pragma unroll
                for (int u = 0; u < (TC_BM * TC_BK / 4) / 128; ++u) {
                    const int o = ct + u * 128;
                    const int r2 = o >> 3, lc = (o & 7) ^ (r2 & 7);
                    const int grow = rt * TC_BM + r2, gcol = (kb_lo + kb) * TC_BK + lc * 4;
                    if (grow < a.rows && gcol < a.n)
                        *reinterpret_cast<float4*>(a.Mout + ((size_t)mat * a.rows + grow) * a.n + gcol) = t0[o];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_stored + 8 * sh);
                if (quarter == 2 && lane == 0) PTC_STAMP(4, kb);
            }
        } else {
        // M = A + B in place and back to HBM; second TF32 term over the tile of B
        for (int kb = grp; kb < KB; kb += 2) {
            const int sh = kb % NH;
            mbar_wait_warp(bar_hfull + 8 * sh, (unsigned)((kb / NH) & 1), a.flags, dead);
            if ((warp & 3) == 2 && lane == 0) PTC_STAMP(1, kb);
            float4* t0 = reinterpret_cast<float4*>(base + (size_t)sh * LONG_BYTES);
            float4* t1 = t0 + A_BYTES / 16;
#pragma unroll
            for (int u = 0; u < (TC_BM * TC_BK / 4) / 128; ++u) {
                const int o = ct + u * 128;             // 16-byte unit of the swizzled tile
                float4 mv = t0[o];
                if (a.has_b) {
                    const float4 e = t1[o];
                    mv.x += e.x; mv.y += e.y; mv.z += e.z; mv.w += e.w;
                    t0[o] = mv;                         // head: M itself (read as TF32 by the tensor core)
                    if (a.Mout) {
                        const int row = o >> 3, lc = (o & 7) ^ (row & 7);      // undo the 128-byte swizzle
                        const int grow = rt * TC_BM + row, gcol = (kb_lo + kb) * TC_BK + lc * 4;
                        if (grow < a.rows && gcol < a.n)
                            *reinterpret_cast<float4*>(a.Mout + ((size_t)mat * a.rows + grow) * a.n + gcol) = mv;
                    }
                }
                const float xs[4] = {mv.x, mv.y, mv.z, mv.w};
                float ms[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float h = __uint_as_float(__float_as_uint(xs[j]) & 0xFFFFE000u);
                    ms[j] = __uint_as_float((__float_as_uint(xs[j] - h) + 0x1000u) & 0xFFFFE000u);   // rounded to nearest TF32
                }
                t1[o] = make_float4(ms[0], ms[1], ms[2], ms[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");    // generic writes -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_conv + 8 * sh);
            if ((warp & 3) == 2 && lane == 0) PTC_STAMP(3, kb);
        }
        }
    } else if (warp == 18) {
        // ---- (pend) issuer of the correction MMAs, a thread of its own so that the projection's issuer does not wait for
        //      them: C_j = P~_prev Qsub_j^T into accumulator j & 1, whose last reader was K block j - 2.  The short-ring stage
        //      it reads is released by the "done" of the projection of the same K block, which cannot be issued before the
        //      converters have consumed C_j. ----
        if (PEND && lane == 0) {
            const unsigned idc3 = tc_idesc(96), idc2 = tc_idesc(64);
            const unsigned long long dPh = tc_smem_desc(pimg_u32), dPm = tc_smem_desc(pimg_u32 + A_BYTES);
            const unsigned long long dS0 = tc_smem_desc(qs_u32), qs_step = PT_QS_BYTES >> 4;
            // images of Qsub: image gi serves the K blocks G gi .. G gi + G - 1, block q at 32 / G floats (8 / G units) into every row
            const int G = a.qs_group, gsh = G == 4 ? 2 : (G == 2 ? 1 : 0);
            const unsigned long long blk_units = 8u >> gsh;
            const int g_lo = kb_lo >> gsh, ngr = ((kb_lo + KB - 1) >> gsh) - g_lo + 1;
            const float* qs_src = a.QSimg + ((size_t)(a.qs_per_node ? mat : qz) * a.qs_groups + g_lo) * (PT_QS_BYTES / 4);
            auto load_group = [&](int gl, int s) {
                mbar_expect_tx(bar_qfull + 8 * s, PT_QS_BYTES);
                bulk_load_1d(qs_u32 + s * PT_QS_BYTES, qs_src + (size_t)gl * (PT_QS_BYTES / 4), PT_QS_BYTES, bar_qfull + 8 * s);
            };
            for (int gl = 0; gl < min(PT_NQ, ngr); ++gl) load_group(gl, gl);
            mbar_wait(bar_pfull, 0u, a.flags, dead);
            int s = 0, phq = 0, gl = 0;             // stage, parity and local index of the current image
            unsigned free_par = 0;                  // bit s: parity of the next completion of qfree[s] to wait for
            for (int j = 0; j < KB; ++j) {
                const int q = (kb_lo + j) & (G - 1), cb = j & 1;
                if (j == 0 || q == 0) mbar_wait_ready(bar_qfull + 8 * s, (unsigned)phq, a.flags, dead);
                if (j >= 2) mbar_wait_ready(bar_cfree + 8 * cb, (unsigned)(((j >> 1) - 1) & 1), a.flags, dead);
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const unsigned long long dS = dS0 + (unsigned long long)s * qs_step + (unsigned long long)q * blk_units;
                const unsigned d_c = tmem_all + (unsigned)(cb * PT_CORR_COLS);
                for (int k = 0; k < a.ksteps; ++k) {
                    const unsigned long long o = (unsigned long long)(2 * k);
                    tc_mma_tf32(d_c, dPh + o, dS + o, idc3, k > 0 ? 1u : 0u);          // h x [h|m|l]
                    tc_mma_tf32(d_c + 32u, dPm + o, dS + o, idc2, 1u);                  // m x [h|m]
                }
                tc_commit(bar_corr + 8 * cb);
                if (q == G - 1 || j == KB - 1) {
                    tc_commit(bar_qfree + 8 * s);           // the image is free once these MMAs have completed
                    // refill the stage that was released one image ago (its MMAs are long done): image gl - 1 + PT_NQ
                    if (gl >= 1 && gl - 1 + PT_NQ < ngr) {
                        const int ps = s == 0 ? PT_NQ - 1 : s - 1;
                        mbar_wait_ready(bar_qfree + 8 * ps, (free_par >> ps) & 1u, a.flags, dead);
                        free_par ^= 1u << ps;
                        load_group(gl - 1 + PT_NQ, ps);
                    }
                    ++gl;
                    if (++s == PT_NQ) { s = 0; phq ^= 1; }
                }
            }
        }
    } else {
        // ---- adders (warps 10-17): accumulators of each K block -> float32 registers; then the epilogue ----
        const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
        const int half = (warp - 10) >> 2;             // which half of the columns this warp adds up
        const int ng = a.Ncp >> 4;                     // 8-column groups per thread
        const unsigned lane_base = (unsigned)(quarter * 32) << 16;
        const unsigned col_base = (unsigned)(half * (a.Ncp >> 1));
        float acc[BT_MAXG][8];
#pragma unroll
        for (int g = 0; g < BT_MAXG; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] = 0.f;
        for (int c = 0; c < KB; ++c) {
            const int hb = c % NB;
            mbar_wait_warp(bar_done + 8 * (c % NH), (unsigned)((c / NH) & 1), a.flags, dead);
            if (warp == 10 && lane == 0) PTC_STAMP(6, c);
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            tc_add_up(acc, tmem, lane_base, col_base, a.Ncp, ng, wide, hb);
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_free + 8 * hb);
            if (warp == 10 && lane == 0) PTC_STAMP(7, c);
        }
        // ---- epilogue: P = registers (+ the small accumulators) ----
        mbar_wait_warp(bar_acc, 0u, a.flags, dead);
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const int row = rt * TC_BM + quarter * 32 + lane;
        float* out = a.P + ((size_t)mat * a.rows + (row < a.rows ? row : 0)) * a.r;
#pragma unroll
        for (int g = 0; g < BT_MAXG; ++g) {
            if (g < ng) {
                float v[8];
                tc_add_small(v, acc[g], tmem, lane_base, col_base, a.Ncp, wide, g);
                if (row < a.rows) {
                    const int j0 = (int)col_base + 8 * g;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j0 + j < a.r) {
                            if (gridDim.z > 1) atomicAdd(out + j0 + j, v[j]);
                            else out[j0 + j] = v[j];
                        }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_all), "r"(ncols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// Back-projection on the tensor cores for more than 16 columns:  Q_i = M_i^T P~  (Algorithm 1:
// Q^(i) <- (Delta^(i))^T P~).  The contraction runs over the rows of M, so the tile of M is the
// MN-major operand: TMA brings 32-row x 32-column boxes of M exactly as they lie in memory (128-byte
// lines, 32-byte swizzle atoms, the one shared-memory form TF32 operands have in this orientation);
// four boxes side by side give the 128 columns of one CTA.  P~^T arrives pre-split and K-major
// (k_split_img_t on P~, three exact terms).  The tile of M is used as two terms: the head is the tile
// itself (read as TF32, i.e. truncated), the second term is x - head rounded to the nearest TF32
// number, written by the converter warps; what is left of x (at most 2^-21 |x|, zero mean) averages
// out over the hundreds of rows of a sum.  Products: h x [h|m|l] and m x [h|m]; m x l is below 2^-32.
// Three shared-memory rings: a deep one for the tiles of M (16 KB stages), a short one for the second
// term of the tile (it lives only from the conversion to the end of the MMAs) and one for the three
// terms of P~^T, one untiled bulk copy per K block of an image in shared-memory order (k_split_img_t);
// the last is requested as many K blocks ahead as it has stages, because the MMAs wait for it.  One mbarrier per K block ("done", by tcgen05.commit) frees both stages and tells
// the adder warps that the accumulators of that K block can be read.
//   up to 80 columns: the three terms of P~^T lie side by side as one B operand of 3 Ncp <= 256 rows:
//     two MMAs per 8 rows (the slow MN-major operand is fetched twice instead of six times); an
//     accumulator set is [head | small | small], sets take turns and are added up in float32
//     registers per K block;
//   above: three MMAs (h x h, h x [m|l], m x [h|m]); the small products keep two accumulators for the
//     whole split, the head product goes through rotating accumulators and float32 registers.
// The rows are dealt to S splits; every split writes its partial [n][r] block, k_reduce_q adds them
// in a fixed order.
// ---------------------------------------------------------------------------------------------
// stages of the short ring
__host__ __device__ inline int back_tc_nm(int Ncp) { return 3 * Ncp <= 256 ? 3 : 2; }
constexpr int BT_NHMAX = 8;       // most stages of the ring of M tiles

struct BackTcArgs {
    float* part;      // [mats][S][n][r]
    int rows, n, r, Ncp, nh, S, kb_per_split;
    int nodes;        // matrices per P~
    int* flags;
    const int* skip;
};

// Stages of the ring of P~^T terms.  Its loads are small but wanted early (the MMAs of a K block cannot start without them)
// and take a full memory latency, so for narrow factors the ring is deeper than the ring of second terms it used to share.
__host__ __device__ inline int back_tc_np(int Ncp) { return Ncp <= 16 ? 8 : (Ncp <= 32 ? 6 : (Ncp <= 48 ? 4 : back_tc_nm(Ncp))); }
__host__ __device__ inline size_t back_tc_fixed_bytes(int Ncp) {
    return (size_t)back_tc_nm(Ncp) * TC_BM * TC_BK * 4 + (size_t)back_tc_np(Ncp) * 3 * Ncp * TC_BK * 4;
}
// stages of the M ring that fit beside the two short rings in 224 KB (0: does not fit)
__host__ __device__ inline int back_tc_nh(int Ncp) {
    const long long left = 224ll * 1024 - 1024 - 512 - (long long)back_tc_fixed_bytes(Ncp);
    const int nh = (int)(left / (TC_BM * TC_BK * 4));
    return nh > BT_NHMAX ? BT_NHMAX : nh;
}
__host__ __device__ inline size_t back_tc_smem_bytes(int Ncp) {
    return (size_t)back_tc_nh(Ncp) * TC_BM * TC_BK * 4 + back_tc_fixed_bytes(Ncp) + 1024 + 512;
}

// shared-memory descriptor of an MN-major TF32 tile: lines of 32 floats along MN, 4-row atoms of 512 bytes along K
// (stride offset), the next 32 floats of MN `mn_block_bytes` further (leading offset); 128-byte swizzle on 32-byte atoms.
__device__ __forceinline__ unsigned long long tc_smem_desc_mn(unsigned addr, unsigned mn_block_bytes) {
    unsigned long long d = 0;
    d |= (unsigned long long)((addr >> 4) & 0x3FFF);
    d |= (unsigned long long)((mn_block_bytes >> 4) & 0x3FFF) << 16;
    d |= (unsigned long long)(512 >> 4) << 32;
    d |= (unsigned long long)1 << 46;
    d |= (unsigned long long)1 << 61;
    return d;
}

__global__ void __launch_bounds__(PT_THREADS, 1)
k_backproject_tc(const __grid_constant__ CUtensorMap tmM, const float* __restrict__ Pimg, BackTcArgs a) {
    extern __shared__ __align__(16) unsigned char bt_smem_raw[];
    if (a.skip && *a.skip) return;
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(bt_smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr unsigned A_BYTES = TC_BM * TC_BK * 4;            // 128 columns x 32 rows
    constexpr unsigned BOX_BYTES = 32 * TC_BK * 4;             // one 32-column box
    const unsigned B_BYTES = (unsigned)a.Ncp * TC_BK * 4;
    const unsigned P_BYTES = 3 * B_BYTES;                      // h, m, l of P~^T of one K block
    const bool wide = 3 * a.Ncp <= 256;
    const int NM = back_tc_nm(a.Ncp), NP = back_tc_np(a.Ncp);
    const int NH = a.nh, NB = wide ? min(4, 512 / (3 * a.Ncp)) : min(3, (512 - 2 * a.Ncp) / a.Ncp);
    unsigned char* short_base = base + (size_t)NH * A_BYTES;             // second terms of the tiles of M: NM stages
    unsigned char* p_base = short_base + (size_t)NM * A_BYTES;           // terms of P~^T: NP stages
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(p_base + (size_t)NP * P_BYTES);
    const unsigned bar_hfull = smem_u32(bars), bar_done = bar_hfull + 8 * NH, bar_bfull = bar_done + 8 * NH;
    const unsigned bar_conv = bar_bfull + 8 * NP, bar_free = bar_conv + 8 * NM, bar_acc = bar_free + 8 * NB;
    unsigned* tmem_slot = reinterpret_cast<unsigned*>(bars + 2 * NH + NP + NM + NB + 1);
    const unsigned ring_u32 = smem_u32(base), short_u32 = smem_u32(short_base), p_u32 = smem_u32(p_base);

    const int ct = blockIdx.x, sp = blockIdx.y, mat = blockIdx.z;
    const int pz = mat / a.nodes;
    const int KBall = (a.rows + TC_BK - 1) / TC_BK;
    const int kb0 = sp * a.kb_per_split;
    const int KB = max(0, min(KBall, kb0 + a.kb_per_split) - kb0);
    unsigned ncols = 32;
    while ((int)ncols < (wide ? NB * 3 : NB + 2) * a.Ncp) ncols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < NH; ++s) { mbar_init(bar_hfull + 8 * s, 1); mbar_init(bar_done + 8 * s, 1); }
        for (int s = 0; s < NP; ++s) mbar_init(bar_bfull + 8 * s, 1);
        for (int s = 0; s < NM; ++s) mbar_init(bar_conv + 8 * s, 8);
        for (int b = 0; b < NB; ++b) mbar_init(bar_free + 8 * b, 8);
        mbar_init(bar_acc, 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(tmem_slot)), "r"(ncols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const unsigned tmem = *tmem_slot;      // wide: set b at 3 b Ncp; else two small accumulators at 0, head b at (2 + b) Ncp
    bool dead = false;
    // K block j is "done" (all its MMAs have completed) in phase j / NH of bar_done[j % NH]
    auto wait_done = [&](int j) { mbar_wait(bar_done + 8 * (j % NH), (unsigned)((j / NH) & 1), a.flags, dead); };

    if (warp == 0) {
        // ---- TMA producer: tiles of M run NH - NP K blocks ahead of the terms of P~^T (one bulk copy per K block) ----
        if (lane == 0) {
            const int lead = max(NH - NP, 0);
            const float* psrc = Pimg + ((size_t)pz * KBall + kb0) * (P_BYTES / 4);
            // (one thread: positions and parities as counters, a non-blocking test before every wait)
            int mj = 0, ms = 0, mph = 1;             // next tile of M: index, stage j % NH, parity of "done" of tile j - NH
            auto issue_m = [&]() {
                if (mj >= NH) mbar_wait_ready(bar_done + 8 * ms, (unsigned)mph, a.flags, dead);
                const unsigned dst = ring_u32 + ms * A_BYTES, bar = bar_hfull + 8 * ms;
                const int row = (kb0 + mj) * TC_BK;
                mbar_expect_tx(bar, A_BYTES);
#pragma unroll
                for (int q = 0; q < 4; ++q) tma_load_3d_sw(dst + q * BOX_BYTES, &tmM, ct * TC_BM + 32 * q, row, mat, bar);
                ++mj;
                if (++ms == NH) { ms = 0; mph ^= 1; }
            };
            for (int j = 0; j < min(lead, KB); ++j) issue_m();
            int ps = 0, ds = 0, dph = 0;             // stage kb % NP; stage and parity of "done" of K block kb - NP
            for (int kb = 0; kb < KB; ++kb) {
                if (mj < KB) issue_m();
                if (kb >= NP) {
                    mbar_wait_ready(bar_done + 8 * ds, (unsigned)dph, a.flags, dead);
                    if (++ds == NH) { ds = 0; dph ^= 1; }
                }
                const unsigned dst = p_u32 + ps * P_BYTES, bar = bar_bfull + 8 * ps;
                mbar_expect_tx(bar, P_BYTES);
                bulk_load_1d(dst, psrc + (size_t)kb * (P_BYTES / 4), P_BYTES, bar);
                if (++ps == NP) ps = 0;
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer (one thread; a second one taking every other K block was measured and changed nothing) ----
        if (lane == 0) {
            const unsigned id1 = tc_idesc(a.Ncp) | (1u << 15);            // bit 15: A is MN-major
            const unsigned id2 = tc_idesc(2 * a.Ncp) | (1u << 15), id3 = tc_idesc(wide ? 3 * a.Ncp : a.Ncp) | (1u << 15);
            // ring positions and parities as counters, descriptors as offsets from those of stage 0
            const unsigned long long dA0 = tc_smem_desc_mn(ring_u32, BOX_BYTES), dM0 = tc_smem_desc_mn(short_u32, BOX_BYTES);
            const unsigned long long dP0 = tc_smem_desc(p_u32);
            const unsigned long long long_step = A_BYTES >> 4, p_step = P_BYTES >> 4, b_off = B_BYTES >> 4;
            int sh = 0, sm = 0, phm = 0, sp_ = 0, php = 0, hb = 0, phb = 1;
            auto advance = [&]() {
                if (++sh == NH) sh = 0;
                if (++sm == NM) { sm = 0; phm ^= 1; }
                if (++sp_ == NP) { sp_ = 0; php ^= 1; }
                if (++hb == NB) { hb = 0; phb ^= 1; }
            };
            for (int kb = 0; kb < KB; ++kb) {
                mbar_wait_ready(bar_conv + 8 * sm, (unsigned)phm, a.flags, dead);
                mbar_wait_ready(bar_bfull + 8 * sp_, (unsigned)php, a.flags, dead);
                if (kb >= NB) mbar_wait_ready(bar_free + 8 * hb, (unsigned)phb, a.flags, dead);   // registers took its last content
                asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
                const unsigned long long dAh = dA0 + (unsigned long long)sh * long_step, dAm = dM0 + (unsigned long long)sm * long_step;
                const unsigned long long dPh = dP0 + (unsigned long long)sp_ * p_step, dPm = dPh + b_off;
                if (wide) {
                    const unsigned d_set = tmem + (unsigned)(3 * hb * a.Ncp);
#pragma unroll
                    for (int k = 0; k < TC_BK / 8; ++k) {
                        const unsigned long long oa = (unsigned long long)(64 * k);   // 8 rows of 128 bytes, in 16-byte units
                        const unsigned long long ob = (unsigned long long)(2 * k);    // 8 floats along the K-major line
                        tc_mma_tf32(d_set, dAh + oa, dPh + ob, id3, k > 0 ? 1u : 0u);                      // h x [h|m|l]
                        tc_mma_tf32(d_set + (unsigned)a.Ncp, dAm + oa, dPh + ob, id2, 1u);                 // m x [h|m]
                    }
                } else {
                    const unsigned d_small = tmem, d_head = tmem + (unsigned)((2 + hb) * a.Ncp);
#pragma unroll
                    for (int k = 0; k < TC_BK / 8; ++k) {
                        const unsigned long long oa = (unsigned long long)(64 * k), ob = (unsigned long long)(2 * k);
                        tc_mma_tf32(d_small, dAh + oa, dPm + ob, id2, (kb > 0 || k > 0) ? 1u : 0u);        // h x [m|l]
                        tc_mma_tf32(d_small, dAm + oa, dPh + ob, id2, 1u);                                 // m x [h|m]
                        tc_mma_tf32(d_head, dAh + oa, dPh + ob, id1, k > 0 ? 1u : 0u);                     // h x h
                    }
                }
                tc_commit(bar_done + 8 * sh);
                advance();
            }
            tc_commit(bar_acc);
        }
    } else if (warp < 10) {
        // ---- converters (warps 2-9): the two lower TF32 terms of the tile of M ----
        const int cv = tid - 64;                       // 0 .. 255
        for (int kb = 0; kb < KB; ++kb) {
            const int sh = kb % NH, sm = kb % NM;
            mbar_wait(bar_hfull + 8 * sh, (unsigned)((kb / NH) & 1), a.flags, dead);
            if (kb >= NM) wait_done(kb - NM);          // the MMAs that read this short stage have completed
            const float4* t0 = reinterpret_cast<const float4*>(base + (size_t)sh * A_BYTES);
            float4* t1 = reinterpret_cast<float4*>(short_base + (size_t)sm * A_BYTES);
#pragma unroll
            for (int u = 0; u < (TC_BM * TC_BK / 4) / 256; ++u) {
                const int o = cv + u * 256;
                const float4 mv = t0[o];
                const float xs[4] = {mv.x, mv.y, mv.z, mv.w};
                float ms[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float h = __uint_as_float(__float_as_uint(xs[j]) & 0xFFFFE000u);
                    ms[j] = __uint_as_float((__float_as_uint(xs[j] - h) + 0x1000u) & 0xFFFFE000u);   // rounded to nearest TF32
                }
                t1[o] = make_float4(ms[0], ms[1], ms[2], ms[3]);
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_conv + 8 * sm);
        }
    } else {
        // ---- adders (warps 10-17): accumulators of each K block -> float32 registers; then the epilogue ----
        const int quarter = warp & 3;                  // tensor-memory lanes this warp may read
        const int half = (warp - 10) >> 2;             // which half of the columns this warp adds up
        const int ng = a.Ncp >> 4;                     // 8-column groups per thread
        const unsigned lane_base = (unsigned)(quarter * 32) << 16;
        const unsigned col_base = (unsigned)(half * (a.Ncp >> 1));
        float acc[BT_MAXG][8];
#pragma unroll
        for (int g = 0; g < BT_MAXG; ++g)
#pragma unroll
            for (int j = 0; j < 8; ++j) acc[g][j] = 0.f;
        for (int c = 0; c < KB; ++c) {
            const int hb = c % NB;
            wait_done(c);
            asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
            tc_add_up(acc, tmem, lane_base, col_base, a.Ncp, ng, wide, hb);
            asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_free + 8 * hb);
        }
        // ---- epilogue: partial Q_i rows of this split = registers (+ the small accumulator) ----
        mbar_wait(bar_acc, 0u, a.flags, dead);
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        const int col = ct * TC_BM + quarter * 32 + lane;
        float* out = a.part + (((size_t)mat * a.S + sp) * a.n + (col < a.n ? col : 0)) * a.r;
#pragma unroll
        for (int g = 0; g < BT_MAXG; ++g) {
            if (g < ng) {
                float v[8];
                tc_add_small(v, acc[g], tmem, lane_base, col_base, a.Ncp, wide, g);
                if (col < a.n) {
                    const int j0 = (int)col_base + 8 * g;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        if (j0 + j < a.r) out[j0 + j] = (KB > 0) ? v[j] : 0.f;
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(ncols) : "memory");
    }
}

}  // namespace psgd
