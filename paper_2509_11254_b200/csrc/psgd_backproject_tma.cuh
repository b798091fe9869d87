// Back-projection Q_i = M_i^T P~ (Algorithm 1: Q^(i) <- Delta^(i)^T P~) for 4, 8 or 16 columns, float32 FMAs, with the tiles
// of M staged by TMA instead of held in registers.
//
// k_backproject keeps the next 8 rows of its 4 columns in registers while it works on the current 8: with the 64 packed
// sums of 16 columns that is 167 registers, three CTAs of 128 threads per multiprocessor and 48 KB of loads in flight,
// which at the memory latency under load is 3.5 TB/s on the whole GPU: the measured rate of that kernel at r = 16 (53 % of
// the copy rate).  Here a thread of the CTA issues 32-row x 256-column tiles (1 KB rows, 32 KB per tile, no swizzle) into a
// three-stage shared-memory ring together with the matching 32 rows of P~ (one untiled bulk copy), two CTAs per
// multiprocessor: 200 KB in flight per multiprocessor, and the registers hold the sums only.  The arithmetic per element is
// unchanged (packed fma.rn.f32x2, P~ rows broadcast from shared memory); the sums of the four row groups of a CTA are added in
// a fixed order.  Every wait is bounded (PSGD_W_TIMEOUT).
#pragma once
#include "psgd_fused.cuh"
#include "psgd_gemm_tc.cuh"

namespace psgd {

constexpr int BQ_THREADS = 256;   // 64 column quads x 4 row groups
constexpr int BQ_ROWS = 32;       // rows per tile
constexpr int BQ_NST = 3;         // tiles in flight per CTA
constexpr unsigned BQ_TILE_BYTES = BQ_ROWS * BP_COLS * 4;

template <int RP>
__host__ __device__ constexpr size_t backq_smem_bytes() {
    return (size_t)BQ_NST * (BQ_TILE_BYTES + BQ_ROWS * RP * 4) + 64 + 128;
}

// Requires r == RP, n % 4 == 0, 16-byte aligned M and P~, rows_per_chunk % 32 == 0, one chunk of columns per matrix.
template <int RP>
__global__ void __launch_bounds__(BQ_THREADS, 2) k_backproject_tma(const __grid_constant__ CUtensorMap tmM, BackArgs a, int* flags) {
    extern __shared__ __align__(16) unsigned char bq_raw[];
    if (a.skip && *a.skip) return;
    unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(bq_raw) + 127) & ~(uintptr_t)127);
    float* ring = reinterpret_cast<float*>(base);                                   // [BQ_NST][32][256]
    float* ps = reinterpret_cast<float*>(base + (size_t)BQ_NST * BQ_TILE_BYTES);    // [BQ_NST][32][RP]
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(ps + BQ_NST * BQ_ROWS * RP);
    const unsigned bar_full = smem_u32(bars), bar_empty = bar_full + 8 * BQ_NST;
    const int tid = threadIdx.x, lane = tid & 31, tx = tid & 63, g = tid >> 6;
    const int col = blockIdx.x * BP_COLS + tx * 4;
    const int s = blockIdx.y, mat = blockIdx.z, c = mat / a.nodes;
    const int n = a.n, r = a.r;
    const int rbeg = s * a.rows_per_chunk, rend = min(a.rows, rbeg + a.rows_per_chunk);
    const int ntiles = (rend - rbeg + BQ_ROWS - 1) / BQ_ROWS;
    const float* Pb = a.Phat + (size_t)c * a.rows * r;

    if (tid == 0) {
        for (int q = 0; q < BQ_NST; ++q) { mbar_init(bar_full + 8 * q, 1); mbar_init(bar_empty + 8 * q, BQ_THREADS / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    // rows of P~ past the end of the matrix are not copied: what the ring holds there must be finite (it meets zeros of M)
    for (int e = tid; e < BQ_NST * BQ_ROWS * RP; e += BQ_THREADS) ps[e] = 0.f;
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    __syncthreads();

    bool dead = false;
    auto issue = [&](int t) {      // thread 0 only
        const int st = t % BQ_NST, row0 = rbeg + t * BQ_ROWS;
        const unsigned pbytes = (unsigned)(min(BQ_ROWS, rend - row0) * RP * 4);
        const unsigned bar = bar_full + 8 * st;
        mbar_expect_tx(bar, BQ_TILE_BYTES + pbytes);
        tma_load_3d(smem_u32(ring + (size_t)st * BQ_ROWS * BP_COLS), &tmM, blockIdx.x * BP_COLS, row0, mat, bar);
        bulk_load_1d(smem_u32(ps + st * BQ_ROWS * RP), Pb + (size_t)row0 * r, pbytes, bar);
    };
    if (tid == 0)
        for (int t = 0; t < min(BQ_NST - 1, ntiles); ++t) issue(t);

    f2p acc2[4][RP / 2];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int k = 0; k < RP / 2; ++k) acc2[j][k] = 0ull;

    for (int t = 0; t < ntiles; ++t) {
        const int st = t % BQ_NST;
        // the tile two ahead goes into the stage the previous tile used: every warp has released it by then
        if (tid == 0 && t + BQ_NST - 1 < ntiles) {
            if (t >= 1) mbar_wait_ready(bar_empty + 8 * ((t - 1) % BQ_NST), (unsigned)(((t - 1) / BQ_NST) & 1), flags, dead);
            issue(t + BQ_NST - 1);
        }
        mbar_wait_ready(bar_full + 8 * st, (unsigned)((t / BQ_NST) & 1), flags, dead);    // (usually there already: a test, no wait)
        const float* tile = ring + (size_t)st * BQ_ROWS * BP_COLS + tx * 4;
        const float* pt = ps + st * BQ_ROWS * RP;
#pragma unroll
        for (int u = 0; u < BQ_ROWS / 4; ++u) {
            const int row = g + 4 * u;
            const float4 v = *reinterpret_cast<const float4*>(tile + row * BP_COLS);
            const float* pr = pt + row * RP;
            const f2p vd[4] = {pack2(v.x, v.x), pack2(v.y, v.y), pack2(v.z, v.z), pack2(v.w, v.w)};
#pragma unroll
            for (int k4 = 0; k4 < RP / 4; ++k4) {
                const ulonglong2 p4 = *reinterpret_cast<const ulonglong2*>(pr + 4 * k4);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    acc2[j][2 * k4 + 0] = ffma2(vd[j], p4.x, acc2[j][2 * k4 + 0]);
                    acc2[j][2 * k4 + 1] = ffma2(vd[j], p4.y, acc2[j][2 * k4 + 1]);
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_empty + 8 * st);
    }
    // sums of the row groups 1..3 through shared memory (the ring is free now), added to group 0's in a fixed order
    __syncthreads();
    float* red = ring;                                          // [3][64][4][RP]
    if (g > 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int k = 0; k < RP; k += 2) {
                const float2 t2 = unpack2(acc2[j][k >> 1]);
                float* d = red + (((size_t)(g - 1) * 64 + tx) * 4 + j) * RP + k;
                d[0] = t2.x; d[1] = t2.y;
            }
    }
    __syncthreads();
    if (g == 0) {
        float* out = a.part + ((size_t)mat * a.S + s) * (size_t)n * r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (col + j < n) {
#pragma unroll
                for (int k = 0; k < RP; k += 2) {
                    const float2 t2 = unpack2(acc2[j][k >> 1]);
                    float s0 = t2.x, s1 = t2.y;
#pragma unroll
                    for (int q = 0; q < 3; ++q) {
                        const float* d = red + (((size_t)q * 64 + tx) * 4 + j) * RP + k;
                        s0 += d[0]; s1 += d[1];
                    }
                    out[(size_t)(col + j) * r + k] = s0;
                    out[(size_t)(col + j) * r + k + 1] = s1;
                }
            }
        }
    }
}

}  // namespace psgd
