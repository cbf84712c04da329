// swift_gemm_static: the skinny weight-streaming GEMM for callers that cannot allocate device memory.
//
// Every other entry point of this library works inside buffers the caller allocated up front.  Some
// callers cannot do even that: code that runs inside somebody else's allocator-controlled process
// (an inference server plug-in that is handed tensors but is forbidden to call cudaMalloc, a callback
// invoked while a stream is being captured, a host thread that must never block on the allocator's
// lock).  For them this file keeps the one piece of scratch memory the split-K GEMM needs — the
// partial-sum slabs and a small control block — in a file-scope device array that is part of the
// library image.  Every GPU that loads the library carries those SWIFT_STATIC_SCRATCH_BYTES until the
// process exits; in exchange the call below touches no allocator at all.
#include "../../include/swift.h"

#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <mutex>
#include <string>

// This translation unit gets its own copies of the shared device code (separate namespace), so that
// nothing here shares a kernel symbol, or a per-kernel attribute, with the rest of the library.
#define swk swk_static
#include "common.cuh"
#include "kernels_gemm_simt.cuh"

using namespace swk;

namespace {

constexpr size_t CONTROL_BYTES = 1024;               // DevState at the front of the array
constexpr int KC = 512;                              // k elements per split: 16 rows x 512 fp32 = 32 KB of shared memory
constexpr int MAX_DEVICES = 64;
static_assert(sizeof(DevState) <= CONTROL_BYTES, "the control block must end before the first partial-sum slab");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is not a
// device address and must never be passed to a kernel.
static __device__ __align__(256) unsigned char g_static_scratch[SWIFT_STATIC_SCRATCH_BYTES];

std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[MAX_DEVICES] = {nullptr};   // device address of g_static_scratch, per device
thread_local std::string g_static_error;

swift_status fail_static(swift_status s, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    g_static_error = buf;
    return s;
}

// Control block for one call: only the row count matters to the GEMM kernel; everything else is zeroed
// so that nothing from an earlier call leaks into this one.
__global__ void static_begin_kernel(DevState* st, int n_rows)
{
    unsigned int* w = reinterpret_cast<unsigned int*>(st);
    for (int i = threadIdx.x; i < (int)(sizeof(DevState) / 4); i += blockDim.x) w[i] = 0u;
    __syncthreads();
    if (threadIdx.x == 0) st->n_rows = n_rows;
}

// y[r][n] = sum over the split-K slabs, in slab order.
__global__ void static_reduce_kernel(const float* __restrict__ part, int n_split, int N, int n_rows, float* __restrict__ y)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x, r = blockIdx.y;
    if (n >= N || r >= n_rows) return;
    float acc = 0.f;
    for (int s = 0; s < n_split; ++s) acc += part[((size_t)s * ROWS + r) * N + n];
    y[(size_t)r * N + n] = acc;
}

template <typename T, int MR>
cudaError_t launch_static(cudaStream_t stream, const DevState* st, const float* x, const T* w, float* part, int N, int K, int S)
{
    dim3 grid((N + GEMM_SIMT_TILE_N - 1) / GEMM_SIMT_TILE_N, S);
    gemm_simt_kernel<T, MR><<<grid, GEMM_SIMT_THREADS, (size_t)MR * KC * sizeof(float), stream>>>(st, x, K, w, part, N, K, KC);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch_static(int n_rows, cudaStream_t stream, const DevState* st, const float* x, const void* w, float* part, int N,
                            int K, int S)
{
    const T* wt = reinterpret_cast<const T*>(w);
    if (n_rows <= 1) return launch_static<T, 1>(stream, st, x, wt, part, N, K, S);
    if (n_rows <= 2) return launch_static<T, 2>(stream, st, x, wt, part, N, K, S);
    if (n_rows <= 4) return launch_static<T, 4>(stream, st, x, wt, part, N, K, S);
    if (n_rows <= 8) return launch_static<T, 8>(stream, st, x, wt, part, N, K, S);
    return launch_static<T, 16>(stream, st, x, wt, part, N, K, S);
}

} // namespace

extern "C" {

const char* swift_gemm_static_error(void) { return g_static_error.c_str(); }

swift_status swift_gemm_static(const void* w_dev, int32_t w_dtype, int32_t N, int32_t K, const float* x_dev, int32_t n_rows,
                               float* y_dev, void* cuda_stream)
{
    if (!w_dev || !x_dev || !y_dev) return fail_static(SWIFT_EINVAL, "null device pointer");
    if (w_dtype != SWIFT_F32 && w_dtype != SWIFT_BF16) return fail_static(SWIFT_EINVAL, "w_dtype must be SWIFT_F32 or SWIFT_BF16");
    if (n_rows < 1 || n_rows > ROWS) return fail_static(SWIFT_ECAPACITY, "n_rows %d outside 1..%d", n_rows, ROWS);
    const int vec = w_dtype == SWIFT_BF16 ? 8 : 4;
    if (N < 1 || K < vec || K % vec) return fail_static(SWIFT_EINVAL, "N >= 1 and K a positive multiple of %d required", vec);
    if (((uintptr_t)w_dev | (uintptr_t)x_dev) % 16) return fail_static(SWIFT_EINVAL, "w_dev and x_dev must be 16-byte aligned");
    const int S = (K + KC - 1) / KC;
    const size_t need = CONTROL_BYTES + (size_t)S * ROWS * (size_t)N * sizeof(float);
    if (need > (size_t)SWIFT_STATIC_SCRATCH_BYTES)
        return fail_static(SWIFT_ECAPACITY,
                           "N = %d, K = %d needs %zu bytes of split-K scratch; the built-in array holds %zu (ceil(K/%d) * 16 * N * 4 + %zu)",
                           N, K, need, (size_t)SWIFT_STATIC_SCRATCH_BYTES, KC, CONTROL_BYTES);
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_static(SWIFT_ECUDA, "cudaGetDevice failed: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= MAX_DEVICES) return fail_static(SWIFT_EUNSUPPORTED, "device ordinal %d not supported", dev);
    unsigned char* base = nullptr;
    {
        // First call on this device: look the array's device address up (with this device current).
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess || !p) return fail_static(SWIFT_ECUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            g_scratch_addr[dev] = static_cast<unsigned char*>(p);
        }
        base = g_scratch_addr[dev];
    }
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    DevState* st = reinterpret_cast<DevState*>(base);
    float* part = reinterpret_cast<float*>(base + CONTROL_BYTES);
    static_begin_kernel<<<1, 128, 0, stream>>>(st, n_rows);
    e = cudaGetLastError();
    if (e == cudaSuccess)
        e = w_dtype == SWIFT_BF16 ? dispatch_static<__nv_bfloat16>(n_rows, stream, st, x_dev, w_dev, part, N, K, S)
                                  : dispatch_static<float>(n_rows, stream, st, x_dev, w_dev, part, N, K, S);
    if (e == cudaSuccess) {
        static_reduce_kernel<<<dim3((N + 255) / 256, n_rows), 256, 0, stream>>>(part, S, N, n_rows, y_dev);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) return fail_static(SWIFT_ECUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return SWIFT_OK;
}

} // extern "C"
