// Kernels of hbf_thermal_step: power map -> explicit Euler substeps of the RC network (Eq. 1) ->
// hotspots and the four-state throttle controller.
//
// The field is kept as the rise above ambient, theta, in float32 with a float32 compensation term per
// cell (Kahan summation of the substep increments): plain float32 accumulation drifts by several mK over
// 10^4..10^5 substeps and stalls once an increment drops under half an ulp of the state.
#include <algorithm>
#include <mutex>
#include <vector>

#include <cooperative_groups.h>

#include "device_utils.cuh"

namespace cg = cooperative_groups;

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

static cudaError_t launch_thermal_generic(const ThermalDev &t, DevState *state, int64_t *pending, int64_t dt_ns, int has_ext,
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


// ======================================================================================================
// The whole step in one launch, for grids that fit the shared memory of one thread-block cluster: eight
// blocks each keep a band of rows of the field (both Jacobi buffers, with one halo row above and below) in
// shared memory and every cell's constants, power and compensation term in registers.  After each substep
// a block writes its first and last row into its neighbours' halo rows through distributed shared memory
// and the cluster barrier separates the substeps.  The arithmetic of a cell is the same, in the same
// order, as in k_euler_substep; the power map is formed by every block for its own cells and the
// hotspots are reduced through block 0.
// ======================================================================================================
constexpr int kThClusterBlocks = 16;                       // blocks of the cluster when the device takes that many (not a portable size), else 8
constexpr int kThClusterPortable = 8;
constexpr int kThThreads = 512;
constexpr int kThCellsPerThread = 8;
constexpr int kThMaxRegions = 1024;

__global__ void __launch_bounds__(kThThreads)
k_thermal_cluster(ThermalDev t, float *theta, DevState *state, int64_t *pending, int64_t dt_ns, int has_ext, float dt_sub,
                  float *temps_out) {
    extern __shared__ __align__(16) unsigned char th_smem[];
    __shared__ double s_region_power[kThMaxRegions];
    __shared__ float s_hot[kThClusterBlocks][3];
    __shared__ float s_part[3][kThThreads / 32];
    cg::cluster_group cluster = cg::this_cluster();
    const uint32_t rank = cluster.block_rank(), n_blocks = cluster.num_blocks();      // (the cluster's size is chosen at launch)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t H = t.H, W = t.W;
    const uint32_t rows = (H + n_blocks - 1) / n_blocks;
    const uint32_t y0 = min(H, rank * rows), y1 = min(H, y0 + rows);
    const uint32_t band_cells = (y1 - y0) * W;
    const uint32_t pitch = (rows + 2) * W;                    // one buffer: halo row, band, halo row
    float *buf0 = reinterpret_cast<float *>(th_smem), *buf1 = buf0 + pitch;

    // power of every region over the window (every block forms the same values), then of this block's cells
    for (uint32_t g = tid; g < t.n_regions; g += kThThreads) {
        double p = 0.0;
        for (int32_t k = t.region_die_ptr[g]; k < t.region_die_ptr[g + 1]; ++k)
            p += ((double)pending[t.region_die_list[k]] * 1e-12) / ((double)dt_ns * 1e-9);
        p += (double)t.region_idle_w[g];
        if (has_ext) p += (double)t.ext_power[g];
        s_region_power[g] = p;
    }
    // field: own rows and the neighbours' boundary rows, from global memory
    for (uint32_t i = tid; i < (y1 - y0 + 2) * W && y1 > y0; i += kThThreads) {
        const uint32_t r = i / W, x = i - r * W;
        const int64_t y = (int64_t)y0 + r - 1;
        buf0[r * W + x] = (y >= 0 && y < (int64_t)H) ? theta[(uint64_t)y * W + x] : 0.0f;
    }
    __syncthreads();
    // this thread's cells: constants, power and compensation in registers
    float kC[kThCellsPerThread], gE[kThCellsPerThread], gW_[kThCellsPerThread], gS[kThCellsPerThread], gN[kThCellsPerThread],
          gs[kThCellsPerThread], P[kThCellsPerThread], cmp[kThCellsPerThread];
    uint32_t off[kThCellsPerThread];
    uint32_t flags[kThCellsPerThread];
#pragma unroll
    for (int c = 0; c < kThCellsPerThread; ++c) {
        const uint32_t li = (uint32_t)c * kThThreads + tid;   // cell of the band, row-major
        flags[c] = 0; off[c] = 0; kC[c] = gE[c] = gW_[c] = gS[c] = gN[c] = gs[c] = P[c] = cmp[c] = 0.0f;
        if (li < band_cells) {
            const uint32_t r = li / W, x = li - r * W, y = y0 + r;
            const uint64_t i = (uint64_t)y * W + x;
            off[c] = (r + 1) * W + x;
            flags[c] = 1u | (x + 1 < W ? 2u : 0u) | (x > 0 ? 4u : 0u) | (y + 1 < H ? 8u : 0u) | (y > 0 ? 16u : 0u);
            kC[c] = dt_sub / t.C[i];
            gE[c] = t.Gx[i]; gW_[c] = x > 0 ? t.Gx[i - 1] : 0.0f; gS[c] = t.Gy[i]; gN[c] = y > 0 ? t.Gy[i - W] : 0.0f;
            gs[c] = t.Gs[i]; cmp[c] = t.comp[i];
            const int32_t g = t.cell_region[i];
            P[c] = g >= 0 ? (float)(s_region_power[g] * (double)t.region_inv_cells[g]) : 0.0f;
        }
    }
    float *upper_halo0 = nullptr, *upper_halo1 = nullptr, *lower_halo0 = nullptr, *lower_halo1 = nullptr;
    if (rank > 0 && y1 > y0) {                                   // the block above: its lower halo row sits after its band
        const uint32_t rows_above = min(H, rank * rows) - min(H, (rank - 1) * rows);
        upper_halo0 = cluster.map_shared_rank(buf0, rank - 1) + (rows_above + 1) * W;
        upper_halo1 = cluster.map_shared_rank(buf1, rank - 1) + (rows_above + 1) * W;
    }
    if (rank + 1 < n_blocks && y1 < H) {                         // the block below: its upper halo row is row 0
        lower_halo0 = cluster.map_shared_rank(buf0, rank + 1);
        lower_halo1 = cluster.map_shared_rank(buf1, rank + 1);
    }
    cluster.sync();
    if (rank == 0) for (uint32_t d = tid; d < t.n_dies; d += kThThreads) pending[d] = 0;   // every block has read it

    float *in = buf0, *out = buf1;
    for (uint32_t k = 0; k < t.n_sub; ++k) {
        float *up = (out == buf0) ? upper_halo0 : upper_halo1, *down = (out == buf0) ? lower_halo0 : lower_halo1;
#pragma unroll
        for (int c = 0; c < kThCellsPerThread; ++c) {
            if (flags[c] & 1u) {
                const uint32_t o = off[c];
                const float Ti = in[o];
                float flow = 0.0f;
                if (flags[c] & 2u)  flow += gE[c] * (Ti - in[o + 1]);
                if (flags[c] & 4u)  flow += gW_[c] * (Ti - in[o - 1]);
                if (flags[c] & 8u)  flow += gS[c] * (Ti - in[o + W]);
                if (flags[c] & 16u) flow += gN[c] * (Ti - in[o - W]);
                const float inc = kC[c] * (P[c] - flow - gs[c] * Ti);
                const float yv = inc - cmp[c];
                const float tn = Ti + yv;
                cmp[c] = (tn - Ti) - yv;
                out[o] = tn;
                const uint32_t r = o / W;                        // first / last row of the band: also the neighbours' halo
                if (r == 1 && up) up[o - W] = tn;
                if (r == y1 - y0 && down) down[o - (y1 - y0) * W] = tn;
            }
        }
        cluster.sync();
        float *tmp = in; in = out; out = tmp;
    }
    // results: field and compensation back to global memory, hotspots to block 0
    float hot[3] = {-INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int c = 0; c < kThCellsPerThread; ++c) {
        if (flags[c] & 1u) {
            const uint32_t li = (uint32_t)c * kThThreads + tid;
            const uint64_t i = (uint64_t)y0 * W + li;
            const float th = in[off[c]];
            theta[i] = th; t.comp[i] = cmp[c];
            const float T = t.ambient_c + th;
            if (temps_out) temps_out[i] = T;
            const int32_t g = t.cell_region[i];
            if (g >= 0) {
                const int32_t kind = t.region_kind[g];
                if (kind == HBF_KIND_HBF) hot[0] = fmaxf(hot[0], T); else if (kind == HBF_KIND_HBM) hot[1] = fmaxf(hot[1], T);
                else if (kind == HBF_KIND_GPU) hot[2] = fmaxf(hot[2], T);
            }
        }
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) {
        for (int o = 16; o > 0; o >>= 1) hot[k] = fmaxf(hot[k], __shfl_xor_sync(0xffffffffu, hot[k], o));
        if (lane == 0) s_part[k][warp] = hot[k];
    }
    __syncthreads();
    if (tid < 3) {
        float v = -INFINITY;
        for (int w = 0; w < kThThreads / 32; ++w) v = fmaxf(v, s_part[tid][w]);
        float *dst = cluster.map_shared_rank(&s_hot[0][0], 0);
        dst[rank * 3 + tid] = v;
    }
    cluster.sync();
    if (rank == 0 && tid == 0) {
        float h[3];
        for (int k = 0; k < 3; ++k) {
            float v = -INFINITY;
            for (uint32_t b = 0; b < n_blocks; ++b) v = fmaxf(v, s_hot[b][k]);
            h[k] = v == -INFINITY ? t.ambient_c : v;
            t.hot[k] = h[k];
        }
        const int mode = next_mode(t, state->mode, quantise_mk(h[0]));
        state->mode = mode;
        if (mode == HBF_MODE_NORMAL) state->q_ppm = 1000000;
        else if (mode == HBF_MODE_LIGHT) state->q_ppm = t.q_light_ppm;
    }
}

static bool thermal_cluster_fits(const ThermalDev &t, int n_blocks, size_t *smem_bytes) {
    const uint32_t rows = (t.H + n_blocks - 1) / n_blocks;
    const size_t smem = (size_t)2 * (rows + 2) * t.W * sizeof(float);
    *smem_bytes = smem;
    return (size_t)rows * t.W <= (size_t)kThThreads * kThCellsPerThread && smem <= 200u * 1024u && t.n_regions <= (uint32_t)kThMaxRegions;
}

// How many blocks the cluster of the one-launch step gets on the current device: 16 where the device can place such a
// cluster (a size beyond the portable 8 has to be allowed per kernel), else 8; 0 when the grid does not fit either.  Asked
// once per (device, shared-memory size) and remembered.
static int thermal_cluster_blocks(const ThermalDev &t, size_t *smem_bytes) {
    struct Entry { int device; size_t smem16; int blocks; };
    static std::mutex mu;
    static std::vector<Entry> known;
    size_t smem16 = 0, smem8 = 0;
    const bool fits16 = thermal_cluster_fits(t, kThClusterBlocks, &smem16), fits8 = thermal_cluster_fits(t, kThClusterPortable, &smem8);
    if (!fits8 && !fits16) return 0;
    int blocks = fits8 ? kThClusterPortable : 0;
    if (fits16) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return blocks;
        std::lock_guard<std::mutex> lock(mu);
        bool found = false;
        for (const Entry &e : known) if (e.device == dev && e.smem16 == smem16) { if (e.blocks) blocks = e.blocks; found = true; break; }
        if (!found) {
            int got = 0;
            if (ensure_dyn_smem((const void *)k_thermal_cluster, smem16) == cudaSuccess &&
                cudaFuncSetAttribute((const void *)k_thermal_cluster, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
                cudaLaunchConfig_t cfg = {};
                cfg.gridDim = dim3(kThClusterBlocks); cfg.blockDim = dim3(kThThreads); cfg.dynamicSmemBytes = smem16;
                cudaLaunchAttribute at[1];
                at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = kThClusterBlocks; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
                cfg.attrs = at; cfg.numAttrs = 1;
                int n = 0;
                if (cudaOccupancyMaxActiveClusters(&n, (const void *)k_thermal_cluster, &cfg) == cudaSuccess && n >= 1) got = kThClusterBlocks;
            }
            (void)cudaGetLastError();                          // a refusal here only means the portable size is used
            known.push_back(Entry{dev, smem16, got});
            if (got) blocks = got;
        }
    }
    *smem_bytes = blocks == kThClusterBlocks ? smem16 : smem8;
    return blocks;
}

cudaError_t launch_thermal_step(const ThermalDev &t, DevState *state, int64_t *pending, int64_t dt_ns, int has_ext,
                                float *d_temps_out, int *cur, int generic_only, cudaStream_t st) {
    const float dt_sub_f = (float)((double)dt_ns * 1e-9 / (double)t.n_sub);
    size_t smem = 0;
    const int blocks = generic_only ? 0 : thermal_cluster_blocks(t, &smem);
    if (blocks) {
        { cudaError_t e = ensure_dyn_smem((const void *)k_thermal_cluster, smem); if (e != cudaSuccess) return e; }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(blocks); cfg.blockDim = dim3(kThThreads); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = blocks; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        float *theta = t.theta[*cur];
        const cudaError_t e = cudaLaunchKernelEx(&cfg, k_thermal_cluster, t, theta, state, pending, dt_ns, has_ext, dt_sub_f, d_temps_out);
        if (e != cudaSuccess) return e;
        g_kernel_launches += 1;
        return cudaGetLastError();
    }
    return launch_thermal_generic(t, state, pending, dt_ns, has_ext, d_temps_out, cur, st);
}

}  // namespace hbf
