// hbf_euler_substeps_static: the explicit-Euler substeps of the package RC network for callers that
// must not allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is off limits -- a host thread between the steps of
// a latency-critical serving loop (cudaMalloc can synchronise the whole device), a plug-in that is
// handed device buffers by its host application and is forbidden to grow the process's footprint, or
// a process whose memory pool has already been handed out in full.  hbf_create / hbf_thermal_step keep
// their ping-pong field in memory that hbf_create allocates; this entry point keeps it in a fixed
// array that is part of the library image instead, so it needs no context and allocates nothing.
//
// The array below lives on every GPU that loads the library, from load until the process exits
// (HBF_STATIC_MAX_CELLS floats = 256 KiB per GPU).  All calls on one GPU share it.
#include <mutex>

#include "hbf_dev.cuh"

namespace {

// Second field buffer of the Jacobi update.  In host code this name is only a handle for the runtime,
// not a device address: kernels get the address that cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) float g_static_field[HBF_STATIC_MAX_CELLS];

constexpr int kMaxDevices = 64;
float *g_field_addr[kMaxDevices] = {};          // per device, filled on the first call on that device
std::mutex g_setup_mutex;

// Same arithmetic, in the same order, as the substep kernel behind hbf_thermal_step.
__global__ void __launch_bounds__(256)
k_euler_substep_static(const float *__restrict__ C, const float *__restrict__ Gx, const float *__restrict__ Gy,
                       const float *__restrict__ Gs, const float *__restrict__ P, const float *__restrict__ th_in,
                       float *__restrict__ th_out, float *__restrict__ comp, uint32_t H, uint32_t W, float dt_sub) {
    const uint32_t x = blockIdx.x * 32 + (threadIdx.x & 31), y = blockIdx.y * 8 + (threadIdx.x >> 5);
    if (x >= W || y >= H) return;
    const uint32_t i = y * W + x;
    const float Ti = th_in[i];
    float flow = 0.0f;
    if (x + 1 < W) flow += Gx[i] * (Ti - th_in[i + 1]);
    if (x > 0)     flow += Gx[i - 1] * (Ti - th_in[i - 1]);
    if (y + 1 < H) flow += Gy[i] * (Ti - th_in[i + W]);
    if (y > 0)     flow += Gy[i - W] * (Ti - th_in[i - W]);
    const float inc = dt_sub / C[i] * (P[i] - flow - Gs[i] * Ti);
    const float yv = inc - comp[i];
    const float tn = Ti + yv;
    comp[i] = (tn - Ti) - yv;
    th_out[i] = tn;
}

__global__ void k_copy_field(const float *__restrict__ src, float *__restrict__ dst, uint32_t n) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = src[i];
}

}  // namespace

extern "C" int hbf_euler_substeps_static(const float *d_cell_C, const float *d_cell_Gx, const float *d_cell_Gy,
                                         const float *d_cell_Gsink, const float *d_cell_power_w, float *d_theta,
                                         float *d_comp, uint32_t grid_h, uint32_t grid_w, uint32_t n_sub,
                                         float dt_sub_s, void *cuda_stream) {
    if (!d_cell_C || !d_cell_Gx || !d_cell_Gy || !d_cell_Gsink || !d_cell_power_w || !d_theta || !d_comp) return HBF_E_INVAL;
    if (grid_h == 0 || grid_w == 0 || n_sub == 0 || !(dt_sub_s > 0.0f)) return HBF_E_INVAL;
    const uint64_t cells = (uint64_t)grid_h * grid_w;
    if (cells > HBF_STATIC_MAX_CELLS) return HBF_E_WORKSPACE;        // the built-in scratch holds HBF_STATIC_MAX_CELLS cells
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HBF_E_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return HBF_E_INVAL;
    float *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_field_addr[dev]) {                                      // once per device, with that device current
            void *p = nullptr;
            if (cudaGetSymbolAddress(&p, g_static_field) != cudaSuccess || !p) return HBF_E_CUDA;
            g_field_addr[dev] = static_cast<float *>(p);
        }
        scratch = g_field_addr[dev];
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const dim3 grid((grid_w + 31) / 32, (grid_h + 7) / 8);
    // Nothing in the scratch has to start at zero: each substep writes every cell of its output field
    // before the next substep reads it, so whatever an earlier call left there is never read.
    float *cur = d_theta, *other = scratch;
    for (uint32_t k = 0; k < n_sub; ++k) {
        k_euler_substep_static<<<grid, 256, 0, st>>>(d_cell_C, d_cell_Gx, d_cell_Gy, d_cell_Gsink, d_cell_power_w, cur, other,
                                                     d_comp, grid_h, grid_w, dt_sub_s);
        float *t = cur; cur = other; other = t;
    }
    if (cur != d_theta)                                                // odd number of substeps: the result sits in the scratch
        k_copy_field<<<(unsigned)((cells + 255) / 256), 256, 0, st>>>(cur, d_theta, (uint32_t)cells);
    hbf::g_kernel_launches += n_sub + (cur != d_theta ? 1u : 0u);
    return cudaGetLastError() == cudaSuccess ? HBF_OK : HBF_E_CUDA;
}
