// Kernels of hbf_thermal_step: power map -> explicit Euler substeps of the RC network (Eq. 1) ->
// hotspots and the four-state throttle controller.
//
// The field is kept as the rise above ambient, theta, in float32 with a float32 compensation term per
// cell (Kahan summation of the substep increments): plain float32 accumulation drifts by several mK over
// 10^4..10^5 substeps and stalls once an increment drops under half an ulp of the state.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

// Power of each region over the window: sum of its dies' energy / dt (pJ/ns = mW), idle and external
// power; then spread evenly over the region's cells.  One thread per region walks that region's dies in
// a fixed order, so the sum is reproducible.  The window's energy is consumed.
__global__ void k_power_map(ThermalDev t, int64_t *pending, int64_t dt_ns, int has_ext) {
    const int tid = threadIdx.x;
    for (uint32_t g = tid; g < t.n_regions; g += blockDim.x) {
        double p = 0.0;
        for (int32_t k = t.region_die_ptr[g]; k < t.region_die_ptr[g + 1]; ++k)
            p += ((double)pending[t.region_die_list[k]] * 1e-12) / ((double)dt_ns * 1e-9);
        p += (double)t.region_idle_w[g];
        if (has_ext) p += (double)t.ext_power[g];
        t.region_power[g] = p;
    }
    __syncthreads();
    const uint32_t nc = t.H * t.W;
    for (uint32_t i = tid; i < nc; i += blockDim.x) {
        const int32_t g = t.cell_region[i];
        t.P[i] = g >= 0 ? (float)(t.region_power[g] * (double)t.region_inv_cells[g]) : 0.0f;
    }
    for (uint32_t d = tid; d < t.n_dies; d += blockDim.x) pending[d] = 0;
}

// One explicit Euler substep, every cell from the previous substep's field (Jacobi).
__global__ void __launch_bounds__(256)
k_euler_substep(ThermalDev t, const float *__restrict__ th_in, float *__restrict__ th_out, float dt_sub) {
    const uint32_t x = blockIdx.x * 32 + (threadIdx.x & 31), y = blockIdx.y * 8 + (threadIdx.x >> 5);
    if (x >= t.W || y >= t.H) return;
    const uint32_t W = t.W, H = t.H, i = y * W + x;
    const float Ti = th_in[i];
    float flow = 0.0f;
    if (x + 1 < W) flow += t.Gx[i] * (Ti - th_in[i + 1]);
    if (x > 0)     flow += t.Gx[i - 1] * (Ti - th_in[i - 1]);
    if (y + 1 < H) flow += t.Gy[i] * (Ti - th_in[i + W]);
    if (y > 0)     flow += t.Gy[i - W] * (Ti - th_in[i - W]);
    const float inc = dt_sub / t.C[i] * (t.P[i] - flow - t.Gs[i] * Ti);
    const float yv = inc - t.comp[i];
    const float tn = Ti + yv;
    t.comp[i] = (tn - Ti) - yv;
    th_out[i] = tn;
}

__device__ __forceinline__ long long quantise_mk(float t_c) { return (long long)floor((double)t_c * 1000.0 + 0.5); }

__device__ __forceinline__ int next_mode(const ThermalDev &t, int mode, long long mk) {
    if (mode == HBF_MODE_SHUTDOWN || mk >= t.shut_mk) return HBF_MODE_SHUTDOWN;
    if (mode == HBF_MODE_NORMAL) return mk >= t.stt_mk ? HBF_MODE_SEVERE : mk >= t.ltt_mk ? HBF_MODE_LIGHT : HBF_MODE_NORMAL;
    if (mode == HBF_MODE_LIGHT) return mk >= t.stt_mk ? HBF_MODE_SEVERE : mk <= t.rtt_mk ? HBF_MODE_NORMAL : HBF_MODE_LIGHT;
    return mk <= t.rtt_mk ? HBF_MODE_NORMAL : mk <= t.ltt_mk ? HBF_MODE_LIGHT : HBF_MODE_SEVERE;
}

// Hottest cell per medium, the controller's transition on the HBF hotspot (quantised to integer mK),
// and the published mode / service fraction for the next batch.
__global__ void __launch_bounds__(1024)
k_controller(ThermalDev t, const float *__restrict__ th, DevState *state, float *temps_out) {
    __shared__ float s_hot[3][32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    float hot[3] = {-INFINITY, -INFINITY, -INFINITY};
    const uint32_t nc = t.H * t.W;
    for (uint32_t i = tid; i < nc; i += blockDim.x) {
        const float T = t.ambient_c + th[i];
        if (temps_out) temps_out[i] = T;
        const int32_t g = t.cell_region[i];
        if (g < 0) continue;
        const int32_t k = t.region_kind[g];
        const int slot = k == HBF_KIND_HBF ? 0 : k == HBF_KIND_HBM ? 1 : k == HBF_KIND_GPU ? 2 : -1;
        if (slot == 0) hot[0] = fmaxf(hot[0], T); else if (slot == 1) hot[1] = fmaxf(hot[1], T); else if (slot == 2) hot[2] = fmaxf(hot[2], T);
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        for (int o = 16; o > 0; o >>= 1) hot[k] = fmaxf(hot[k], __shfl_xor_sync(0xffffffffu, hot[k], o));
        if (lane == 0) s_hot[k][warp] = hot[k];
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            float v = lane < (int)(blockDim.x >> 5) ? s_hot[k][lane] : -INFINITY;
            for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
            hot[k] = v == -INFINITY ? t.ambient_c : v;
        }
        if (lane == 0) {
            t.hot[0] = hot[0]; t.hot[1] = hot[1]; t.hot[2] = hot[2];
            const int mode = next_mode(t, state->mode, quantise_mk(hot[0]));
            state->mode = mode;
            if (mode == HBF_MODE_NORMAL) state->q_ppm = 1000000;
            else if (mode == HBF_MODE_LIGHT) state->q_ppm = t.q_light_ppm;
        }
    }
}

cudaError_t launch_thermal_step(const ThermalDev &t, DevState *state, int64_t *pending, int64_t dt_ns, int has_ext,
                                float *d_temps_out, int *cur, cudaStream_t st) {
    k_power_map<<<1, 1024, 0, st>>>(t, pending, dt_ns, has_ext);
    const float dt_sub = (float)((double)dt_ns * 1e-9 / (double)t.n_sub);
    dim3 grid((t.W + 31) / 32, (t.H + 7) / 8);
    int c = *cur;
    for (uint32_t k = 0; k < t.n_sub; ++k) {
        k_euler_substep<<<grid, 256, 0, st>>>(t, t.theta[c], t.theta[c ^ 1], dt_sub);
        c ^= 1;
    }
    *cur = c;
    g_kernel_launches += 2ull + t.n_sub;
    k_controller<<<1, 1024, 0, st>>>(t, t.theta[c], state, d_temps_out);
    return cudaGetLastError();
}

}  // namespace hbf
