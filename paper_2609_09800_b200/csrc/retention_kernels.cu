// Retention, refresh and wear (Design D4) as data-parallel kernels.
//   per epoch (hbf_retention_advance): region temperatures -> Arrhenius damage rate per region -> damage and
//     eligibility per block -> the refresh plan.  The paper's emission order (eligibility epoch, channel round
//     robin, die round robin, zone, block, page) is not walked: every quantum computes its own place in it.  With
//     r_die the quantum's rank in its die's (zone, plane, block, page) list, the dies of a channel served in turn
//     put it at r_ch = sum over the channel's dies d' of min(len[d'], r_die), plus the dies before its own that
//     still have a quantum of that rank; the channels served in turn put it at the same expression over channels
//     with r_ch.  The ranks come from one scan per die; the rest is arithmetic on the per-die lengths.
//   per batch (hbf_submit_batch): the claim window finds the batch index below which the modeled accesses claim
//     one outstanding quantum each (they claim in index order), before the batch is served; after it, the reads
//     are counted into their blocks' disturb counters, blocks whose last quantum is now claimed commit, and the
//     claimed energy is booked on the claimants' dies.
//   idle time (hbf_retention_decay) drains quanta on an account of its own and commits likewise.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

__device__ __forceinline__ bool ret_ready(const RangeSnap &rs, const hbf_access_t *acc, uint64_t i, uint64_t *off, uint32_t *bytes, uint32_t *op) {
    const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
    const uint64_t addr = __ldg(rec), bf = __ldg(rec + 2);
    const int64_t issue = (int64_t)__ldg(rec + 1);
    int g = 0;
    if (classify(rs, addr, issue, (uint32_t)bf, (uint32_t)(bf >> 32), &g) != HBF_ST_READY) return false;
    if (off) *off = rs.media_offset[g] + (addr - rs.base[g]);
    if (bytes) *bytes = (uint32_t)bf;
    if (op) *op = (uint32_t)(bf >> 32) & 1u;
    return true;
}

__device__ __forceinline__ void load_ranges(RangeSnap *dst, const RangeSnap *src) {
    for (int i = threadIdx.x; i < (int)(sizeof(RangeSnap) / 4); i += blockDim.x)
        reinterpret_cast<uint32_t *>(dst)[i] = reinterpret_cast<const uint32_t *>(src)[i];
}

// inclusive scan of one value per thread over the block; *total (nullable) receives the sum
template <int THREADS>
__device__ __forceinline__ uint32_t block_scan_incl(uint32_t v, uint32_t *total) {
    __shared__ uint32_t s_w[THREADS / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const uint32_t y = __shfl_up_sync(0xffffffffu, x, o); if (lane >= o) x += y; }
    __syncthreads();                                          // the previous use of s_w is over
    if (lane == 31) s_w[warp] = x;
    __syncthreads();
    uint32_t before = 0, sum = 0;
    for (int w = 0; w < THREADS / 32; ++w) { const uint32_t t = s_w[w]; if (w < warp) before += t; sum += t; }
    if (total) *total = sum;
    return x + before;
}

// =====================================================================================================
// claim window: how far into the batch do the outstanding quanta reach?
// =====================================================================================================
constexpr int kRetTile = 1024;
constexpr int kRetWinThreads = 256;

// Tiles are handed out in order from a counter; a block stops taking tiles once the tiles already finished hold at
// least as many modeled accesses as there is debt (the tiles in flight only add to that).  Work is proportional
// to the reach of the debt, not to the batch.
__global__ void __launch_bounds__(kRetWinThreads)
k_ret_window(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges_g, RetDev r) {
    __shared__ RangeSnap rs;
    __shared__ uint32_t s_tile, s_cnt;
    RetState *st = r.st;
    const unsigned long long debt = st->planned - st->claimed - st->decayed;
    if (debt == 0ull || n == 0ull) return;
    load_ranges(&rs, ranges_g);
    const uint64_t n_tiles = (n + kRetTile - 1) / kRetTile;
    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) {
            s_cnt = 0u;
            const unsigned long long seen = atomicAdd(&st->counted, 0ull);
            s_tile = seen >= debt ? 0xffffffffu : (uint32_t)min(atomicAdd(&st->tickets, 1ull), 0xffffffffull);
        }
        __syncthreads();
        const uint64_t tile = s_tile;
        if (tile >= n_tiles) break;
        uint32_t c = 0;
#pragma unroll
        for (int k = 0; k < kRetTile / kRetWinThreads; ++k) {
            const uint64_t i = tile * kRetTile + (uint64_t)k * kRetWinThreads + threadIdx.x;
            if (i < n && ret_ready(rs, acc, i, nullptr, nullptr, nullptr)) ++c;
        }
        c = (uint32_t)warp_sum((long long)c);
        if (lane_id() == 0 && c) atomicAdd(&s_cnt, c);
        __syncthreads();
        if (threadIdx.x == 0) { r.tile_count[tile] = s_cnt; __threadfence(); atomicAdd(&st->counted, (unsigned long long)s_cnt); }
    }
}

// One block: the tile in which the running count reaches the debt, then the record inside it.
__global__ void __launch_bounds__(kRetTile)
k_ret_find(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges_g, RetDev r) {
    __shared__ RangeSnap rs;
    __shared__ unsigned long long s_base, s_before;
    __shared__ uint32_t s_found;
    RetState *st = r.st;
    const int tid = threadIdx.x;
    const unsigned long long debt = st->planned - st->claimed - st->decayed;
    if (debt == 0ull || n == 0ull) {
        if (tid == 0) { st->claim_limit = 0ull; st->claims_now = 0ull; st->tickets = 0ull; st->counted = 0ull; }
        return;
    }
    load_ranges(&rs, ranges_g);
    const uint64_t n_tiles = (n + kRetTile - 1) / kRetTile;
    const uint64_t T = min((uint64_t)st->tickets, n_tiles);
    if (tid == 0) { s_base = 0ull; s_found = 0xffffffffu; }
    __syncthreads();
    for (uint64_t chunk = 0; chunk < T; chunk += kRetTile) {
        const uint64_t t = chunk + (uint64_t)tid;
        const uint32_t v = t < T ? r.tile_count[t] : 0u;
        uint32_t sum = 0;
        const uint32_t incl = block_scan_incl<kRetTile>(v, &sum);
        const unsigned long long base = s_base;
        if (t < T && base + incl >= debt && base + incl - v < debt) { s_found = (uint32_t)t; s_before = base + incl - v; }
        __syncthreads();
        if (s_found != 0xffffffffu) break;
        if (tid == 0) s_base = base + sum;
        __syncthreads();
    }
    const uint32_t found = s_found;
    if (found == 0xffffffffu) {                               // the whole batch claims and debt remains
        if (tid == 0) { st->claim_limit = n; st->claims_now = s_base; }
    } else {
        const uint32_t need = (uint32_t)(debt - s_before);    // 1 .. the tile's count
        const uint64_t i = (uint64_t)found * kRetTile + (uint64_t)tid;
        const uint32_t flag = (i < n && ret_ready(rs, acc, i, nullptr, nullptr, nullptr)) ? 1u : 0u;
        const uint32_t incl = block_scan_incl<kRetTile>(flag, nullptr);
        if (flag && incl == need) { st->claim_limit = i + 1ull; st->claims_now = debt; }
    }
    if (tid == 0) { st->tickets = 0ull; st->counted = 0ull; }
}

cudaError_t launch_ret_window(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const RetDev &r, int sm_count, cudaStream_t st) {
    const uint64_t tiles = (n + kRetTile - 1) / kRetTile;
    const unsigned grid = (unsigned)std::max<uint64_t>(1, std::min<uint64_t>(tiles, (uint64_t)sm_count * 4));
    k_ret_window<<<grid, kRetWinThreads, 0, st>>>(acc, n, ranges, r);
    k_ret_find<<<1, kRetTile, 0, st>>>(acc, n, ranges, r);
    g_kernel_launches += 2;
    return cudaGetLastError();
}

// =====================================================================================================
// after the batch: read disturb, commits, bookkeeping
// =====================================================================================================
// The in-order serve pass counts the reads into the disturb counters as it streams the batch (observed_inline).  This
// pass covers the other cases: the batch was served without that pass (count now), or the pass ran and the batch was
// then refused (take the counts back: the same reads, the same amounts).
__global__ void __launch_bounds__(256)
k_ret_observe(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges_g,
              const ModelParams *__restrict__ mp_g, const hbf_batch_result_t *result, RetDev r) {
    __shared__ RangeSnap rs;
    __shared__ ModelParams mp;
    const bool ok = result->code == HBF_OK, inline_done = r.st->observed_inline != 0u;
    if (ok == inline_done) return;                           // counted and accepted, or neither
    const bool undo = inline_done;
    load_ranges(&rs, ranges_g);
    for (int i = threadIdx.x; i < (int)(sizeof(ModelParams) / 4); i += blockDim.x)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    __syncthreads();
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
        uint64_t off; uint32_t bytes, op;
        if (!ret_ready(rs, acc, i, &off, &bytes, &op) || op) continue;
        const uint64_t in_page = off & ((1ull << mp.page_shift) - 1ull);
        const uint32_t npages = (uint32_t)((in_page + bytes + (1ull << mp.page_shift) - 1ull) >> mp.page_shift);
        atomicAdd(&r.disturb[ret_block_of(mp, r, off)], undo ? 0u - npages : npages);
    }
}

// a block whose last quantum lies below the watermark commits one cycle and clears its counters
__global__ void __launch_bounds__(256)
k_ret_commit(const hbf_batch_result_t *result, RetDev r) {
    RetState *st = r.st;
    unsigned long long mark = st->claimed + st->decayed;
    if (result) { if (result->code != HBF_OK) return; mark += st->claims_now; }
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < r.n_blocks; b += stride) {
        if (r.epoch_of[b] == 0u || r.last_pos[b] >= mark) continue;
        const uint32_t pec = r.pec[b] + 1u;
        r.pec[b] = pec; r.damage[b] = 0.0; r.disturb[b] = 0u; r.epoch_of[b] = 0u;
        atomicAdd(&st->commits, 1ull);
        if (pec >= r.max_pec) { r.worn[b] = 1; atomicAdd(&st->worn_blocks, 1ull); }
    }
}

__global__ void k_ret_close(const hbf_batch_result_t *result, int64_t *pending, int64_t quantum_pj, uint32_t n_dies, RetDev r) {
    const bool ok = result->code == HBF_OK;
    for (uint32_t d = threadIdx.x; d < n_dies; d += blockDim.x) {
        const uint32_t c = r.die_claims[d];
        if (ok && c) pending[d] += (int64_t)c * quantum_pj;
        r.die_claims[d] = 0u;
    }
    if (threadIdx.x == 0) {
        RetState *st = r.st;
        if (ok) st->claimed += st->claims_now;
        st->claims_now = 0ull; st->claim_limit = 0ull; st->observed_inline = 0u;
    }
}

static unsigned ret_grid(uint64_t items, int sm_count) {
    return (unsigned)std::max<uint64_t>(1, std::min<uint64_t>((items + 255) / 256, (uint64_t)sm_count * 8));
}

cudaError_t launch_ret_close(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev, const ModelParams &mp,
                             const hbf_batch_result_t *result, int64_t *pending, int binned, const RetDev &r, int sm_count, cudaStream_t st) {
    if (n) k_ret_observe<<<ret_grid(n, sm_count), 256, 0, st>>>(acc, n, ranges, mp_dev, result, r);
    k_ret_commit<<<ret_grid(r.n_blocks, sm_count), 256, 0, st>>>(result, r);
    const int64_t page = (int64_t)1 << mp.page_shift;
    const int64_t quantum_pj = mp.e_cmd_read_pj + mp.e_byte_read_pj * page + mp.e_cmd_prog_pj + mp.e_byte_prog_pj * page;
    k_ret_close<<<1, 256, 0, st>>>(result, pending, binned ? 0 : quantum_pj, mp.n_dies, r);   // with the time bins on, the ledger has it
    g_kernel_launches += n ? 3 : 2;
    return cudaGetLastError();
}

// =====================================================================================================
// one epoch: temperatures -> damage -> eligibility -> plan
// =====================================================================================================
__device__ __forceinline__ int ordered_int(float f) { const int k = __float_as_int(f); return k >= 0 ? k : k ^ 0x7fffffff; }
__device__ __forceinline__ float ordered_float(int k) { return __int_as_float(k >= 0 ? k : k ^ 0x7fffffff); }

__global__ void k_ret_region_clear(RetDev r) {
    for (uint32_t g = threadIdx.x; g < r.n_regions; g += blockDim.x) r.region_max[g] = ordered_int(-INFINITY);
}
__global__ void __launch_bounds__(256)
k_ret_region_max(const float *__restrict__ theta, const int32_t *__restrict__ cell_region, uint64_t n_cells, RetDev r) {
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_cells; i += stride) {
        const int32_t g = cell_region[i];
        if (g >= 0) atomicMax(&r.region_max[g], ordered_int(theta[i]));
    }
}

// Arrhenius lifetime at each region's temperature (first equation of D4) and the damage it adds per block in this
// epoch (second equation of D4); opens the epoch
__global__ void k_ret_rate(RetDev r, int from_field, float ambient_c, double dt_s) {
    for (uint32_t g = threadIdx.x; g < r.n_regions; g += blockDim.x) {
        double temp_c;
        if (from_field) {
            const float rise = ordered_float(r.region_max[g]);
            temp_c = rise == -INFINITY ? (double)ambient_c : (double)(ambient_c + rise);
        } else {
            temp_c = r.region_temp[g];
        }
        const double life = r.l_ref_s * exp(r.ea_over_kb * (1.0 / (temp_c + 273.15) - 1.0 / r.t_ref_k));
        r.rate[g] = r.accel * dt_s / life;
    }
    if (threadIdx.x == 0) r.st->epoch += 1u;
}

__global__ void __launch_bounds__(256)
k_ret_damage(RetDev r, const int32_t *__restrict__ die_region, uint32_t blocks_per_die) {
    const uint32_t epoch = r.st->epoch;
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    for (uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; b < r.n_blocks; b += stride) {
        if (r.worn[b]) continue;
        const uint32_t g = die_region ? (uint32_t)die_region[b / blocks_per_die] : 0u;
        const double d = r.damage[b] + r.rate[g];
        r.damage[b] = d;
        if (r.epoch_of[b] == 0u && (d >= r.lead || (r.disturb_limit && r.disturb[b] >= r.disturb_limit))) r.epoch_of[b] = epoch;
    }
}

// one thread block per die: rank of every newly eligible block in the die's (zone, plane, block) order
constexpr int kRetRankThreads = 256;
__global__ void __launch_bounds__(kRetRankThreads)
k_ret_rank(RetDev r, uint32_t planes) {
    const uint32_t epoch = r.st->epoch, die = blockIdx.x;
    const uint32_t per_die = planes * r.bpp, zone_span = planes * r.bpz;
    uint32_t running = 0;
    for (uint32_t o0 = 0; o0 < per_die; o0 += kRetRankThreads) {
        const uint32_t o = o0 + threadIdx.x;
        uint64_t b = 0; uint32_t flag = 0;
        if (o < per_die) {
            const uint32_t zone = o / zone_span, rem = o % zone_span, pl = rem / r.bpz, kk = rem % r.bpz;
            b = ((uint64_t)die * planes + pl) * r.bpp + zone * r.bpz + kk;
            flag = r.epoch_of[b] == epoch ? 1u : 0u;
        }
        uint32_t sum = 0;
        const uint32_t incl = block_scan_incl<kRetRankThreads>(flag, &sum);
        if (flag) r.rank[b] = running + incl - 1u;
        running += sum;
    }
    if (threadIdx.x == 0) r.die_len[die] = (unsigned long long)running * r.ppb;
}

__global__ void k_ret_chan(RetDev r, uint32_t channels, uint32_t dies) {
    __shared__ unsigned long long s_total;
    if (threadIdx.x == 0) s_total = 0ull;
    __syncthreads();
    for (uint32_t c = threadIdx.x; c < channels; c += blockDim.x) {
        unsigned long long s = 0;
        for (uint32_t d = 0; d < dies; ++d) s += r.die_len[c * dies + d];
        r.chan_len[c] = s;
        atomicAdd(&s_total, s);
    }
    __syncthreads();
    if (threadIdx.x == 0) r.st->epoch_total = s_total;
    // For the plan kernel: the lengths in ascending order with their running sums, and for every channel the lengths of
    // the channels before it in ascending order.  With them the place of a quantum among the channels, a sum of
    // min(length, x) over all channels and a count of longer channels before its own, takes two binary searches
    // instead of a pass over the channels.  (Every length, and their sum, is below 2^32.)
    if (r.chan_tab) {
        uint32_t *sorted = r.chan_tab, *run = r.chan_tab + channels, *before = r.chan_tab + 2 * channels + 1;
        for (uint32_t c = threadIdx.x; c < channels; c += blockDim.x) {
            const unsigned long long lc = r.chan_len[c];
            uint32_t at = 0;
            for (uint32_t j = 0; j < channels; ++j) { const unsigned long long lj = r.chan_len[j]; at += (lj < lc || (lj == lc && j < c)) ? 1u : 0u; }
            sorted[at] = (uint32_t)lc;
        }
        for (uint32_t k = threadIdx.x; k < channels * channels; k += blockDim.x) {
            const uint32_t ch = k / channels, c = k % channels;      // channel c among the channels before ch
            if (c >= ch) continue;
            const unsigned long long lc = r.chan_len[c];
            uint32_t at = 0;
            for (uint32_t j = 0; j < ch; ++j) { const unsigned long long lj = r.chan_len[j]; at += (lj < lc || (lj == lc && j < c)) ? 1u : 0u; }
            before[(size_t)ch * channels + at] = (uint32_t)lc;
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t sum = 0;
            for (uint32_t k = 0; k < channels; ++k) { run[k] = sum; sum += sorted[k]; }
            run[channels] = sum;
        }
    }
}

// how many of the n ascending values at tab are at most x
__device__ __forceinline__ uint32_t count_at_most(const uint32_t *__restrict__ tab, uint32_t n, uint32_t x) {
    uint32_t lo = 0, len = n;
    while (len > 0u) {
        const uint32_t half = len >> 1;
        if (__ldg(tab + lo + half) <= x) { lo += half + 1u; len -= half + 1u; } else len = half;
    }
    return lo;
}

// one warp per block, its lanes over the block's pages.  Every length and rank of an epoch is below 2^32 (a quantum id
// is 32 bits and a block is planned at most once at a time), so the arithmetic is 32-bit.
__global__ void __launch_bounds__(256)
k_ret_emit(RetDev r, uint32_t channels, uint32_t dies, uint32_t planes) {
    const RetState *st = r.st;
    const uint32_t epoch = st->epoch;
    const unsigned long long base = st->planned;
    const uint64_t base_mod = base % r.plan_cap;
    const uint32_t blocks_per_die = planes * r.bpp;
    const int lane = threadIdx.x & 31;
    const uint64_t warps = ((uint64_t)gridDim.x * blockDim.x) >> 5;
    for (uint64_t b = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; b < r.n_blocks; b += warps) {
        if (r.epoch_of[b] != epoch) continue;
        const uint32_t die = (uint32_t)(b / blocks_per_die), ch = die / dies, di = die % dies;
        const uint32_t first = r.rank[b] * r.ppb;
        const unsigned long long *dlen = r.die_len + (size_t)ch * dies;
        for (uint32_t pg = (uint32_t)lane; pg < r.ppb; pg += 32u) {
            const uint32_t r_die = first + pg;
            uint32_t r_ch = 0;
            for (uint32_t d = 0; d < dies; ++d) {
                const uint32_t len = (uint32_t)__ldg(dlen + d);
                r_ch += min(len, r_die) + ((d < di && len > r_die) ? 1u : 0u);
            }
            uint32_t pos = 0;
            if (r.chan_tab) {
                const uint32_t k = count_at_most(r.chan_tab, channels, r_ch);                       // channels no longer than r_ch: all of theirs
                pos = __ldg(r.chan_tab + channels + k) + r_ch * (channels - k);                       // the others: r_ch each
                pos += ch - count_at_most(r.chan_tab + 2 * channels + 1 + (size_t)ch * channels, ch, r_ch);   // and one more of every longer channel before this one
            } else {
                for (uint32_t c = 0; c < channels; ++c) {
                    const uint32_t len = (uint32_t)__ldg(r.chan_len + c);
                    pos += min(len, r_ch) + ((c < ch && len > r_ch) ? 1u : 0u);
                }
            }
            uint64_t slot = base_mod + pos;
            if (slot >= r.plan_cap) slot -= r.plan_cap;
            r.plan[slot] = (uint32_t)(b * r.ppb + pg);
            if (pg + 1u == r.ppb) r.last_pos[b] = base + pos;       // the last page's place: a block's pages go out in order
        }
    }
}

__global__ void k_ret_epoch_close(RetDev r) { r.st->planned += r.st->epoch_total; r.st->epoch_total = 0ull; }

cudaError_t launch_ret_advance(const RetDev &r, const ModelParams &mp, const ThermalDev *field, const float *theta, const int32_t *die_region,
                               int have_temps, int64_t dt_ns, int sm_count, cudaStream_t st) {
    const int from_field = have_temps ? 0 : 1;
    float ambient = 0.0f;
    if (from_field) {
        const uint64_t cells = (uint64_t)field->H * field->W;
        ambient = field->ambient_c;
        k_ret_region_clear<<<1, 256, 0, st>>>(r);
        k_ret_region_max<<<ret_grid(cells, sm_count), 256, 0, st>>>(theta, field->cell_region, cells, r);
        g_kernel_launches += 2;
    }
    k_ret_rate<<<1, 256, 0, st>>>(r, from_field, ambient, (double)dt_ns * 1e-9);
    k_ret_damage<<<ret_grid(r.n_blocks, sm_count), 256, 0, st>>>(r, die_region, mp.planes * r.bpp);
    k_ret_rank<<<mp.n_dies, kRetRankThreads, 0, st>>>(r, mp.planes);
    k_ret_chan<<<1, 256, 0, st>>>(r, mp.channels, mp.dies);
    k_ret_emit<<<ret_grid(r.n_blocks * 32, sm_count), 256, 0, st>>>(r, mp.channels, mp.dies, mp.planes);
    k_ret_epoch_close<<<1, 1, 0, st>>>(r);
    g_kernel_launches += 6;
    return cudaGetLastError();
}

// =====================================================================================================
// idle time drains debt: one quantum per scaled quantum time (Eq. 3), on an account of its own
// =====================================================================================================
__global__ void k_ret_decay(RetDev r, const DevState *state, int64_t quantum_ns, int64_t idle_ns) {
    RetState *st = r.st;
    const int64_t q = state->q_ppm;
    const int64_t scaled = q == 1000000 ? quantum_ns : (quantum_ns * 1000000 + q - 1) / q;
    unsigned long long drained = (unsigned long long)(idle_ns / scaled);
    const unsigned long long debt = st->planned - st->claimed - st->decayed;
    st->decayed += min(drained, debt);
}

cudaError_t launch_ret_decay(const RetDev &r, const ModelParams &mp, const DevState *state, int64_t idle_ns, int sm_count, cudaStream_t st) {
    k_ret_decay<<<1, 1, 0, st>>>(r, state, mp.t_read_ns + mp.t_prog_ns, idle_ns);
    k_ret_commit<<<ret_grid(r.n_blocks, sm_count), 256, 0, st>>>(nullptr, r);
    g_kernel_launches += 2;
    return cudaGetLastError();
}

}  // namespace hbf
