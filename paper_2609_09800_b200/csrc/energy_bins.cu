// Time-bin power integration (Section "Design", event-based energy model).  The ledger keeps energy per (bin, die);
// an event longer than one bin contributes to each bin it touches by the fraction of its duration spent there.
// Here the event of an access is its array service interval [start, start + s) on its die; shares are
// whole pJ, floor(E * overlap / s), and the event's last bin takes what is left.  The ledger is a ring of bins
// that starts at the bin the thermal clock stands in; time before it is booked into that bin, time past the
// ring's end into the ring's last bin.  Integer adds in any order: the result does not depend on scheduling.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

__device__ __forceinline__ void ledger_add(unsigned long long *ledger, uint32_t n_dies, uint32_t n_bins, int64_t cur_bin,
                                           uint32_t die, int64_t bin, int64_t pj) {
    bin = max(bin, cur_bin);
    bin = min(bin, cur_bin + (int64_t)n_bins - 1);
    if (pj) atomicAdd(&ledger[(size_t)(bin % (int64_t)n_bins) * n_dies + die], (unsigned long long)pj);
}

// one event: energy pj over [start, start + s), split over the bins it overlaps.  Every bin before the event's last one
// gets floor(pj * overlap / s); the overlap is a whole bin for all of them but the first, so the bins that the ring clamps
// into its first or last slot are booked in one step each and the loop only walks bins inside the ring: at most n_bins
// turns, whatever the ratio of service time to bin width.
__device__ __forceinline__ void ledger_event(unsigned long long *ledger, uint32_t n_dies, uint32_t n_bins, int64_t cur_bin, int64_t bin_ns,
                                             uint32_t die, int64_t start, int64_t s, int64_t pj) {
    const int64_t end = start + s;
    const int64_t b0 = start / bin_ns, b1 = (end - 1) / bin_ns;
    if (b0 == b1) { ledger_add(ledger, n_dies, n_bins, cur_bin, die, b0, pj); return; }
    const int64_t ring_hi = cur_bin + (int64_t)n_bins - 1;
    const int64_t first = (int64_t)(((unsigned __int128)(uint64_t)pj * (uint64_t)((b0 + 1) * bin_ns - start)) / (uint64_t)s);
    const int64_t full = (int64_t)(((unsigned __int128)(uint64_t)pj * (uint64_t)bin_ns) / (uint64_t)s);
    auto run = [&](int64_t from, int64_t to) {               // shares of the bins [from, to), from >= b0, to <= b1
        return to <= from ? (int64_t)0 : (from == b0 ? first + (to - from - 1) * full : (to - from) * full);
    };
    const int64_t below_end = min(b1, max(b0, cur_bin));     // bins [b0, below_end) lie before the ring
    const int64_t above_begin = min(b1, max(below_end, ring_hi));   // bins [above_begin, b1) lie at or past its last slot
    int64_t given = 0;
    const int64_t below = run(b0, below_end);
    ledger_add(ledger, n_dies, n_bins, cur_bin, die, cur_bin, below); given += below;
    for (int64_t b = below_end; b < above_begin; ++b) {
        const int64_t share = b == b0 ? first : full;
        ledger_add(ledger, n_dies, n_bins, cur_bin, die, b, share); given += share;
    }
    const int64_t above = run(above_begin, b1);
    ledger_add(ledger, n_dies, n_bins, cur_bin, die, ring_hi, above); given += above;
    ledger_add(ledger, n_dies, n_bins, cur_bin, die, b1, pj - given);
}

// Runs after the batch's results are final: start = completion - (a read's transfer) - service.  With retention on, an
// access below the claim limit served a refresh quantum first: that is an event of its own, ahead of the access's.
__global__ void __launch_bounds__(256)
k_energy_bins(const hbf_access_t *__restrict__ acc, uint64_t n, const int64_t *__restrict__ completion,
              const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp_g, const BatchCtrl *__restrict__ ctrl,
              const hbf_batch_result_t *__restrict__ result, unsigned long long *ledger, int64_t bin_ns, uint32_t n_bins,
              int64_t cur_bin, const unsigned long long *claim_limit_p, int64_t quantum_pj) {
    __shared__ ModelParams mp;
    if (result->code != HBF_OK) return;                      // a refused batch books nothing
    for (int i = threadIdx.x; i < (int)(sizeof(ModelParams) / 4); i += blockDim.x)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    __syncthreads();
    const RangeSnap &rs = *ranges;
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const uint32_t n_dies = mp.n_dies;
    const uint64_t claim_limit = claim_limit_p ? *claim_limit_p : 0ull;
    const int64_t quantum_ns = q_ppm == 1000000 ? mp.t_read_ns + mp.t_prog_ns
        : (int64_t)div64((uint64_t)(mp.t_read_ns + mp.t_prog_ns) * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
        const uint64_t addr = __ldg(rec), bf = __ldg(rec + 2);
        const int64_t issue = (int64_t)__ldg(rec + 1);
        const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
        int g = 0;
        if (classify(rs, addr, issue, bytes, flags, &g) != HBF_ST_READY) continue;
        const Decoded d = decode(mp, rs.media_offset[g] + (addr - rs.base[g]), bytes);
        const uint32_t op = flags & 1u;
        const Terms t = service_terms(mp, bytes, d.npages, op, q_ppm, div_q);
        const int64_t end = completion[i] - (op ? 0 : t.xfer);
        int64_t start = end - t.s;
        if (i < claim_limit) {
            ledger_event(ledger, n_dies, n_bins, cur_bin, bin_ns, d.die, start - quantum_ns, quantum_ns, quantum_pj);
        }
        ledger_event(ledger, n_dies, n_bins, cur_bin, bin_ns, d.die, start, t.s, t.energy);
    }
}

// the thermal step takes the bin the clock stands in
__global__ void k_take_bin(unsigned long long *row, int64_t *pending, uint32_t n_dies) {
    const uint32_t d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d < n_dies) { pending[d] += (int64_t)row[d]; row[d] = 0ull; }
}

cudaError_t launch_energy_bins(const hbf_access_t *acc, uint64_t n, const int64_t *completion, const RangeSnap *ranges,
                               const ModelParams *mp_dev, const BatchCtrl *ctrl, const hbf_batch_result_t *result,
                               unsigned long long *ledger, int64_t bin_ns, uint32_t n_bins, int64_t cur_bin, int sm_count,
                               const unsigned long long *claim_limit, int64_t quantum_pj, cudaStream_t st) {
    if (n == 0) return cudaSuccess;
    const unsigned grid = (unsigned)std::min<uint64_t>((n + 255) / 256, (uint64_t)std::max(1, sm_count) * 8);
    k_energy_bins<<<grid, 256, 0, st>>>(acc, n, completion, ranges, mp_dev, ctrl, result, ledger, bin_ns, n_bins, cur_bin, claim_limit, quantum_pj);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_take_bin(unsigned long long *row, int64_t *pending, uint32_t n_dies, cudaStream_t st) {
    k_take_bin<<<(n_dies + 255) / 256, 256, 0, st>>>(row, pending, n_dies);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

}  // namespace hbf
