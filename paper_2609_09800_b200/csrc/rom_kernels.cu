// Reduced-order thermal model at run time (Eq. 2): x' = A x + B p + b, T = C x + D p + d, x the state before the
// update.  A few hundred states: one thread block steps the model, a warp per row of the matrices, in double
// (the matrices come from a fit in double; at this size the arithmetic is not what a step costs).
#include "hbf_dev.cuh"

namespace hbf {

constexpr int kRomThreads = 512;

__global__ void __launch_bounds__(kRomThreads)
k_rom_steps(uint32_t n, uint32_t m, uint32_t o, const double *__restrict__ A, const double *__restrict__ B,
            const double *__restrict__ b, const double *__restrict__ C, const double *__restrict__ D,
            const double *__restrict__ d, double *x, const double *__restrict__ power, uint32_t n_steps,
            double *__restrict__ temps_out) {
    extern __shared__ double rom_smem[];                     // x [n], x' [n], p [m]
    double *xs = rom_smem, *xn = rom_smem + n, *ps = rom_smem + 2 * n;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = kRomThreads / 32;
    for (uint32_t i = tid; i < n; i += kRomThreads) xs[i] = x[i];
    __syncthreads();
    for (uint32_t k = 0; k < n_steps; ++k) {
        for (uint32_t j = tid; j < m; j += kRomThreads) ps[j] = power[(size_t)k * m + j];
        __syncthreads();
        for (uint32_t row = warp; row < n + o; row += n_warps) {          // rows of [A B] first, then rows of [C D]
            const bool out_row = row >= n;
            const uint32_t r = out_row ? row - n : row;
            const double *mx = out_row ? C + (size_t)r * n : A + (size_t)r * n;
            const double *mp = out_row ? D + (size_t)r * m : B + (size_t)r * m;
            double acc = 0.0;
            for (uint32_t j = lane; j < n; j += 32) acc += mx[j] * xs[j];
            for (uint32_t j = lane; j < m; j += 32) acc += mp[j] * ps[j];
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
            if (lane == 0) {
                if (out_row) temps_out[(size_t)k * o + r] = acc + d[r];
                else xn[r] = acc + b[r];
            }
        }
        __syncthreads();
        for (uint32_t i = tid; i < n; i += kRomThreads) xs[i] = xn[i];
        __syncthreads();
    }
    for (uint32_t i = tid; i < n; i += kRomThreads) x[i] = xs[i];
}

cudaError_t launch_rom_steps(uint32_t n, uint32_t m, uint32_t o, const double *A, const double *B, const double *b,
                             const double *C, const double *D, const double *d, double *x, const double *power,
                             uint32_t n_steps, double *temps_out, cudaStream_t st) {
    const size_t smem = (size_t)(2 * n + m) * sizeof(double);
    k_rom_steps<<<1, kRomThreads, smem, st>>>(n, m, o, A, B, b, C, D, d, x, power, n_steps, temps_out);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

}  // namespace hbf
