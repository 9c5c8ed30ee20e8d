// Reduced-order thermal model at run time (Eq. 2): x' = A x + B p + b, T = C x + D p + d, x the state before the
// update.  A few hundred states: one thread block steps the model, a warp per row of the matrices, in double
// (the matrices come from a fit in double; at this size the arithmetic is not what a step costs).
#include <cooperative_groups.h>

#include "hbf_dev.cuh"

namespace cg = cooperative_groups;

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

// The same steps on a cluster of eight blocks: block c keeps rows [c * rpc, (c + 1) * rpc) of [A B; C D] in its shared
// memory for the whole launch, computes those rows every step and writes its part of x' into the next-state buffer of
// all eight blocks through distributed shared memory; one cluster barrier per step.  Each row is summed in the same
// order as in the single-block kernel, so both give the same bits.
constexpr int kRomClusterBlocks = 8;
constexpr int kRomClusterThreads = 256;

__global__ void __cluster_dims__(kRomClusterBlocks, 1, 1) __launch_bounds__(kRomClusterThreads)
k_rom_steps_cluster(uint32_t n, uint32_t m, uint32_t o, uint32_t rpc, const double *__restrict__ A, const double *__restrict__ B,
                    const double *__restrict__ b, const double *__restrict__ C, const double *__restrict__ D,
                    const double *__restrict__ d, double *x, const double *__restrict__ power, uint32_t n_steps,
                    double *__restrict__ temps_out) {
    extern __shared__ double rom_smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank();
    const uint32_t width = n + m;
    double *rows = rom_smem;                                 // [rpc][n + m]: this block's rows of [A B] then [C D]
    double *bias = rows + (size_t)rpc * width;               // [rpc]
    double *xb0 = bias + rpc, *xb1 = xb0 + n, *ps = xb1 + n; // state, next state, this step's power
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, n_warps = kRomClusterThreads / 32;
    const uint32_t row0 = rank * rpc, row1 = min(n + o, row0 + rpc);
    for (uint32_t r = row0 + warp; r < row1; r += n_warps) {
        const bool out_row = r >= n;
        const uint32_t rr = out_row ? r - n : r;
        const double *mx = out_row ? C + (size_t)rr * n : A + (size_t)rr * n;
        const double *mp = out_row ? D + (size_t)rr * m : B + (size_t)rr * m;
        double *dst = rows + (size_t)(r - row0) * width;
        for (uint32_t j = lane; j < n; j += 32) dst[j] = mx[j];
        for (uint32_t j = lane; j < m; j += 32) dst[n + j] = mp[j];
        if (lane == 0) bias[r - row0] = out_row ? d[rr] : b[rr];
    }
    for (uint32_t i = tid; i < n; i += kRomClusterThreads) xb0[i] = x[i];
    double *cur = xb0, *nxt = xb1;
    cluster.sync();
    for (uint32_t k = 0; k < n_steps; ++k) {
        for (uint32_t j = tid; j < m; j += kRomClusterThreads) ps[j] = power[(size_t)k * m + j];
        __syncthreads();
        for (uint32_t r = row0 + warp; r < row1; r += n_warps) {
            const double *mr = rows + (size_t)(r - row0) * width;
            double acc = 0.0;
            for (uint32_t j = lane; j < n; j += 32) acc += mr[j] * cur[j];
            for (uint32_t j = lane; j < m; j += 32) acc += mr[n + j] * ps[j];
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
            const double v = acc + bias[r - row0];
            if (r >= n) { if (lane == 0) temps_out[(size_t)k * o + (r - n)] = v; }
            else if (lane < kRomClusterBlocks) cluster.map_shared_rank(nxt, lane)[r] = v;    // every block's copy of x'
        }
        cluster.sync();                                      // x' is complete everywhere; nobody reads x any more
        double *t = cur; cur = nxt; nxt = t;
    }
    if (rank == 0)
        for (uint32_t i = tid; i < n; i += kRomClusterThreads) x[i] = cur[i];
}

// ---- the thermal step of a context on a reduced-order model: power vector, one model step, controller --------
// Power of each region over the window, as the grid's power map computes it (one thread per region walks its dies in
// a fixed order): the model's input vector.  The window's energy is consumed.
__global__ void k_rom_power(ThermalDev t, int64_t *pending, int64_t dt_ns, int has_ext, double *__restrict__ p_out) {
    for (uint32_t g = threadIdx.x; g < t.n_regions; g += blockDim.x) {
        double p = 0.0;
        for (int32_t k = t.region_die_ptr[g]; k < t.region_die_ptr[g + 1]; ++k)
            p += ((double)pending[t.region_die_list[k]] * 1e-12) / ((double)dt_ns * 1e-9);
        p += (double)t.region_idle_w[g];
        if (has_ext) p += (double)t.ext_power[g];
        p_out[g] = p;
    }
    __syncthreads();
    for (uint32_t d = threadIdx.x; d < t.n_dies; d += blockDim.x) pending[d] = 0;
}

__device__ __forceinline__ int rom_next_mode(const ThermalDev &t, int mode, long long mk) {
    if (mode == HBF_MODE_SHUTDOWN || mk >= t.shut_mk) return HBF_MODE_SHUTDOWN;
    if (mode == HBF_MODE_NORMAL) return mk >= t.stt_mk ? HBF_MODE_SEVERE : mk >= t.ltt_mk ? HBF_MODE_LIGHT : HBF_MODE_NORMAL;
    if (mode == HBF_MODE_LIGHT) return mk >= t.stt_mk ? HBF_MODE_SEVERE : mk <= t.rtt_mk ? HBF_MODE_NORMAL : HBF_MODE_LIGHT;
    return mk <= t.rtt_mk ? HBF_MODE_NORMAL : mk <= t.ltt_mk ? HBF_MODE_LIGHT : HBF_MODE_SEVERE;
}

// hottest output of each medium, the controller's transition on the HBF one (quantised to integer mK)
__global__ void k_rom_controller(ThermalDev t, const double *__restrict__ temps, const int32_t *__restrict__ kind, uint32_t n_out,
                                 DevState *state) {
    if (threadIdx.x != 0) return;
    double hot[3] = {-1e300, -1e300, -1e300};
    for (uint32_t i = 0; i < n_out; ++i) {
        const int slot = kind[i] == HBF_KIND_HBF ? 0 : kind[i] == HBF_KIND_HBM ? 1 : kind[i] == HBF_KIND_GPU ? 2 : -1;
        if (slot >= 0 && temps[i] > hot[slot]) hot[slot] = temps[i];
    }
    for (int k = 0; k < 3; ++k) { if (hot[k] == -1e300) hot[k] = (double)t.ambient_c; t.hot[k] = (float)hot[k]; }
    const int mode = rom_next_mode(t, state->mode, (long long)floor(hot[0] * 1000.0 + 0.5));
    state->mode = mode;
    if (mode == HBF_MODE_NORMAL) state->q_ppm = 1000000;
    else if (mode == HBF_MODE_LIGHT) state->q_ppm = t.q_light_ppm;
}

cudaError_t launch_rom_power(const ThermalDev &t, int64_t *pending, int64_t dt_ns, int has_ext, double *p_out, cudaStream_t st) {
    k_rom_power<<<1, 256, 0, st>>>(t, pending, dt_ns, has_ext, p_out);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_rom_controller(const ThermalDev &t, const double *temps, const int32_t *kind, uint32_t n_out, DevState *state,
                                  cudaStream_t st) {
    k_rom_controller<<<1, 32, 0, st>>>(t, temps, kind, n_out, state);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

static size_t rom_cluster_smem(uint32_t n, uint32_t m, uint32_t o, uint32_t *rpc_out) {
    const uint32_t rpc = (n + o + kRomClusterBlocks - 1) / kRomClusterBlocks;
    *rpc_out = rpc;
    return ((size_t)rpc * (n + m) + rpc + 2 * (size_t)n + m) * sizeof(double);
}

cudaError_t launch_rom_steps(uint32_t n, uint32_t m, uint32_t o, const double *A, const double *B, const double *b,
                             const double *C, const double *D, const double *d, double *x, const double *power,
                             uint32_t n_steps, double *temps_out, cudaStream_t st) {
    uint32_t rpc = 0;
    const size_t csmem = rom_cluster_smem(n, m, o, &rpc);
    if (csmem <= 200u * 1024u) {                             // the rows fit the shared memory of eight blocks
        { cudaError_t e = ensure_dyn_smem((const void *)k_rom_steps_cluster, csmem); if (e != cudaSuccess) return e; }
        k_rom_steps_cluster<<<kRomClusterBlocks, kRomClusterThreads, csmem, st>>>(n, m, o, rpc, A, B, b, C, D, d, x, power, n_steps, temps_out);
        g_kernel_launches += 1;
        return cudaGetLastError();
    }
    const size_t smem = (size_t)(2 * n + m) * sizeof(double);
    k_rom_steps<<<1, kRomThreads, smem, st>>>(n, m, o, A, B, b, C, D, d, x, power, n_steps, temps_out);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

}  // namespace hbf
