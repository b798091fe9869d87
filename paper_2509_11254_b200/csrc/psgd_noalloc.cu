// psgd_backproject_static: the back-projection Q_i = M_i^T P~ and its node mean for callers
// that cannot allocate device memory.  The row-chunk partial sums, which the handle-based
// path keeps in the caller's workspace, live here in a fixed file-scope device array.
//
// This file is compiled as part of psgd_api.cu's translation unit (it is #included there),
// so the array, the one-time address lookup and the launches below share one file.
#include <mutex>

namespace {

// Scratch for the partial sums: [N][S][n][r] floats, S = number of row chunks.  Every GPU
// that loads the library holds these PSGD_STATIC_SCRATCH_BYTES until the process exits.
static __device__ __align__(256) float g_static_scratch[PSGD_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

// In host code `g_static_scratch` is only a stand-in for the symbol, not a device address;
// the address a kernel can use has to be asked for, once per device, with that device current.
psgd_status static_scratch_for_current_device(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PSGD_E_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) return PSGD_E_CUDA;
        g_scratch_addr[dev] = static_cast<float*>(p);
    }
    *out = g_scratch_addr[dev];
    return PSGD_OK;
}

template <int RP>
void static_back_launch(BackArgs a, int mats, bool vec, cudaStream_t st) {
    a.nchunks = ceil_div(a.r, RP);
    dim3 grid(ceil_div(a.n, BP_COLS), a.S, mats * a.nchunks);
    if (vec) k_backproject<RP, 4><<<grid, BP_THREADS, 0, st>>>(a);
    else k_backproject<RP, 1><<<grid, BP_THREADS, 0, st>>>(a);
}

}  // namespace

extern "C" psgd_status psgd_backproject_static(const float* M, const float* P_hat, float* Q_node, float* Q_mean,
                                               int64_t m, int64_t n, int r, int N, psgd_stream stream) {
    if (!M || !P_hat || !Q_mean) return PSGD_E_NULL;
    if (!(m >= n && n >= r && r >= 1 && r <= MAX_R && N >= 1 && N <= 65535 && m <= (1 << 24))) return PSGD_E_INVALID;
    const size_t max_floats = PSGD_STATIC_SCRATCH_BYTES / sizeof(float);
    const size_t per_chunk = (size_t)N * (size_t)n * (size_t)r;  // floats of partial sums per row chunk
    if (per_chunk > max_floats) return PSGD_E_TOO_LARGE;
    float* scratch = nullptr;
    psgd_status s = static_scratch_for_current_device(&scratch);
    if (s != PSGD_OK) return s;

    // row chunking: as many chunks as fill the GPU, but no more than the scratch holds
    const int colblk = ceil_div(n, BP_COLS);
    int64_t base = (int64_t)N * colblk;
    int S = (int)std::max<int64_t>(1, (8 * (int64_t)device_sms() + base - 1) / base);
    S = std::min<int64_t>(S, ceil_div(m, BP_SUB));
    S = (int)std::min<size_t>((size_t)S, max_floats / per_chunk);
    int rpc = (int)align_up(ceil_div(m, S), BP_SUB);
    S = ceil_div(m, rpc);

    cudaStream_t st = (cudaStream_t)stream;
    BackArgs a{M, P_hat, scratch, (int)m, (int)n, r, N, 1, rpc, S};
    bool vec = (n % 4 == 0) && aligned16(M);
    // every partial that k_reduce_q reads below is written by this launch, so nothing
    // left over from an earlier call is ever summed and no clearing pass is needed
    if (r <= 4) static_back_launch<4>(a, N, vec, st);
    else if (r <= 8) static_back_launch<8>(a, N, vec, st);
    else static_back_launch<16>(a, N, vec, st);
    size_t tot = (size_t)n * r;
    k_reduce_q<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(scratch, Q_node, Q_mean, (int)n, r, N, S, 1);
    return cudaGetLastError() == cudaSuccess ? PSGD_OK : PSGD_E_CUDA;
}
