// Kernels of hbf_submit_batch, sort path:
//   begin -> classify (load, range filter, decode, key) -> plan -> histogram -> onesweep radix passes ->
//   scan (segmented max-plus scan with decoupled look-back, fused with the scatter back to batch order
//   and the per-die reductions) -> finish (commit or refuse).
// Every kernel reads the batch control block first and does nothing once the batch is refused, so the
// whole sequence can be enqueued without a host round trip.
#include <algorithm>
#include <mutex>
#include <vector>

#include "device_utils.cuh"

namespace hbf {

// =====================================================================================================
// begin: snapshot mode and q (before any reservation, Eq. 3), stage the queue state, clear the block
// =====================================================================================================
// role 0: first kernel of a batch; run_sort tells whether the sort path serves it.
// role 1: placed between the in-order attempt and the sort kernels; it starts the batch over for the
//         sort path when the in-order attempt found the records out of issue order, else does nothing.
__global__ void k_begin(BatchCtrl *ctrl, const DevState *state, const int64_t *busy, int64_t *busy_stage,
                        hbf_die_stats_t *stats_stage, uint32_t *hist, uint32_t n_queues, uint32_t n_dies,
                        int role, int run_sort, uint32_t *die_claims) {
    const int tid = threadIdx.x;
    if (role == 1) {
        if (ctrl->skip || !ctrl->run_sort) return;
        run_sort = 1;
    }
    __syncthreads();
    uint32_t *w = reinterpret_cast<uint32_t *>(ctrl);
    for (int i = tid; i < (int)(sizeof(BatchCtrl) / 4); i += blockDim.x) w[i] = 0u;
    __syncthreads();
    if (tid == 0) {
        int32_t mode = state->mode;
        ctrl->mode = mode; ctrl->q_ppm = state->q_ppm;
        ctrl->div_q = make_div64((uint64_t)state->q_ppm);
        ctrl->key_and = ~0ull;
        ctrl->run_sort = (uint32_t)run_sort;
        if (state->poisoned) { ctrl->code = HBF_E_TIMEOUT; ctrl->skip = 1; }
        else if (mode == HBF_MODE_SHUTDOWN) { ctrl->code = HBF_E_LINK_SHUTDOWN; ctrl->skip = 1; }
        else if (mode == HBF_MODE_SEVERE) { ctrl->code = HBF_E_THROTTLED; ctrl->skip = 1; }
    }
    for (uint32_t r = tid; r < n_queues; r += blockDim.x) busy_stage[r] = busy[r];
    int64_t *s = reinterpret_cast<int64_t *>(stats_stage);
    for (uint32_t i = tid; i < n_dies * 6u; i += blockDim.x) s[i] = 0;
    for (int i = tid; i < kMaxPasses * kRadix; i += blockDim.x) hist[i] = 0u;
    if (die_claims)                                          // retention on: an in-order attempt that was handed over counted some
        for (uint32_t d = tid; d < n_dies; d += blockDim.x) die_claims[d] = 0u;
}

// =====================================================================================================
// classify: 16-byte coalesced loads of the 24-byte records into shared memory, then per record the
// range filter, the decode and the sort key (queue << 47 | issue).  NATIVE rows are answered here.
// =====================================================================================================
constexpr int kClsThreads = 256;
constexpr int kClsItems = 4;
constexpr int kClsTile = kClsThreads * kClsItems;       // 1024 records = 24 KiB

// (four resident blocks per SM: 1.96 -> 1.40 ms at 200 M against three at 84 registers; six was slower)
__global__ void __launch_bounds__(kClsThreads, 4)
k_classify(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges_g,
           const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl, uint64_t *__restrict__ keys, uint64_t *__restrict__ terms,
           uint8_t *__restrict__ status, int64_t *__restrict__ completion, int64_t *__restrict__ stall) {
    __shared__ RangeSnap rs;
    __shared__ ModelParams mp;
    __shared__ __align__(16) uint64_t rec[kClsTile * 3];
    if (ctrl->skip || !ctrl->run_sort) return;
    const int tid = threadIdx.x;
    for (int i = tid; i < (int)(sizeof(RangeSnap) / 4); i += kClsThreads)
        reinterpret_cast<uint32_t *>(&rs)[i] = reinterpret_cast<const uint32_t *>(ranges_g)[i];
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kClsThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    const bool aligned16 = (reinterpret_cast<uintptr_t>(acc) & 15u) == 0;
    const uint64_t sentinel = (uint64_t)mp_g->n_queues << kIssueBits;

    unsigned long long n_native = 0, n_ready = 0, n_fault = 0, k_or = 0, k_and = ~0ull;
    unsigned unsorted = 0;
    const uint64_t n_tiles = (n + kClsTile - 1) / kClsTile;
    for (uint64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const uint64_t base = tile * kClsTile;
        const int cnt = (int)min((uint64_t)kClsTile, n - base);
        __syncthreads();
        const uint64_t *src = reinterpret_cast<const uint64_t *>(acc + base);
        if (cnt == kClsTile && aligned16) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
            uint4 *d4 = reinterpret_cast<uint4 *>(rec);
#pragma unroll
            for (int k = 0; k < kClsTile * 24 / 16 / kClsThreads; ++k) d4[tid + k * kClsThreads] = __ldg(s4 + tid + k * kClsThreads);
        } else {
            for (int i = tid; i < cnt * 3; i += kClsThreads) rec[i] = __ldg(src + i);
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kClsItems; ++k) {
            const int li = tid + k * kClsThreads;
            if (li >= cnt) break;
            const uint64_t i = base + li;
            const uint64_t addr = rec[li * 3];
            const int64_t issue = (int64_t)rec[li * 3 + 1];
            const uint64_t bf = rec[li * 3 + 2];
            const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
            int64_t prev;
            if (li > 0) prev = (int64_t)rec[li * 3 - 2];
            else prev = i > 0 ? acc[i - 1].issue_ns : INT64_MIN;
            unsorted |= (issue < prev) ? 1u : 0u;
            int g = 0;
            const int st = classify(rs, addr, issue, bytes, flags, &g);
            uint64_t key = sentinel;
            if (st == HBF_ST_READY) {
                const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
                const Decoded d = decode(mp, off, bytes);
                key = ((uint64_t)d.queue << kIssueBits) | (uint64_t)issue;
                terms[i] = (uint64_t)bytes | ((uint64_t)(flags & 1u) << 32) | ((uint64_t)d.npages << 33);   // (fewer than 2^31 pages)
                ++n_ready;
            } else if (st == HBF_ST_NATIVE) {
                ++n_native;
                completion[i] = issue; stall[i] = 0;
            } else {
                ++n_fault;
            }
            keys[i] = key;
            k_or |= key; k_and &= key;
            if (status) status[i] = (uint8_t)st;
        }
    }
    n_native = (unsigned long long)warp_sum((long long)n_native);
    n_ready = (unsigned long long)warp_sum((long long)n_ready);
    n_fault = (unsigned long long)warp_sum((long long)n_fault);
    k_or = warp_or(k_or); k_and = warp_and(k_and);
    unsorted = __any_sync(0xffffffffu, unsorted);
    if (lane_id() == 0) {
        if (n_native) atomicAdd(&ctrl->n_native, n_native);
        if (n_ready) atomicAdd(&ctrl->n_ready, n_ready);
        if (n_fault) atomicAdd(&ctrl->n_fault, n_fault);
        atomicOr(&ctrl->key_or, k_or); atomicAnd(&ctrl->key_and, k_and);
        if (unsorted) atomicOr(&ctrl->unsorted, 1u);
    }
}

// =====================================================================================================
// plan: refuse the batch on any fail-closed access; otherwise choose the radix passes.  Only bits that
// differ between keys take part; a batch already in issue order needs the queue bits only (the sort is
// stable, so issue order and then batch index survive as the minor keys).
// =====================================================================================================
__device__ __forceinline__ uint64_t compact_key(uint64_t key, uint32_t lo_bits, uint32_t hi_bits) {
    const uint64_t lo = lo_bits ? (key & ((1ull << lo_bits) - 1ull)) : 0ull;
    const uint64_t hi = (key >> kIssueBits) & ((1ull << hi_bits) - 1ull);
    return lo | (hi << lo_bits);
}

// The digit of one pass straight from the key: the digit's bits lie in the issue field, in the queue field, or (one pass
// at most) in both; two shifts and two masks instead of compacting the whole key first.
struct DigitSel { uint32_t sh_lo, m_lo, sh_hi, m_hi, up; uint64_t raw; };      // raw: the digit's bits where they lie in the key
__device__ __forceinline__ DigitSel digit_sel(const SortPlan &p, int pass) {
    const uint32_t shift = p.shift[pass], bits = p.bits[pass];
    const uint32_t n_lo = shift < p.lo_bits ? min(bits, p.lo_bits - shift) : 0u, n_hi = bits - n_lo;
    DigitSel d;
    d.sh_lo = n_lo ? shift : 0u; d.m_lo = (1u << n_lo) - 1u;
    d.sh_hi = n_hi ? (max(shift, p.lo_bits) - p.lo_bits) + (uint32_t)kIssueBits : 0u; d.m_hi = (1u << n_hi) - 1u;
    d.up = n_lo;
    d.raw = ((uint64_t)d.m_lo << d.sh_lo) | ((uint64_t)d.m_hi << d.sh_hi);
    return d;
}
__device__ __forceinline__ uint32_t digit_at(uint64_t key, const DigitSel &d) {
    return ((uint32_t)(key >> d.sh_lo) & d.m_lo) | (((uint32_t)(key >> d.sh_hi) & d.m_hi) << d.up);
}

__global__ void k_plan(BatchCtrl *ctrl, int force_full) {
    if (threadIdx.x != 0 || ctrl->skip || !ctrl->run_sort) return;
    if (ctrl->n_fault) { ctrl->code = HBF_E_ACCESS_FAULT; ctrl->skip = 1; return; }
    const uint64_t diff = ctrl->key_or ^ ctrl->key_and;
    const uint64_t dlo = diff & kIssueMask, dhi = diff >> kIssueBits;
    uint32_t lo = (ctrl->unsorted || force_full) ? (dlo ? 64u - (uint32_t)__clzll((long long)dlo) : 0u) : 0u;
    uint32_t hi = dhi ? 64u - (uint32_t)__clzll((long long)dhi) : 0u;
    const uint32_t total = lo + hi;
    const uint32_t np = (total + 7u) / 8u;
    SortPlan p; p.n_passes = np; p.lo_bits = lo; p.hi_bits = hi;
    uint32_t shift = 0;
    for (uint32_t i = 0; i < (uint32_t)kMaxPasses; ++i) {
        uint32_t b = 0;
        if (i < np) b = total / np + (i < total % np ? 1u : 0u);
        p.shift[i] = shift; p.bits[i] = b; shift += b;
    }
    ctrl->plan = p;
}

// =====================================================================================================
// histogram of the first pass's digit (shared-memory bins).  The later passes' histograms are counted by the pass before
// each, which has the keys in registers anyway: six shared-memory adds per key in one kernel took 1.8 ms at 200 M.
// =====================================================================================================
constexpr int kHistThreads = 512;

__global__ void __launch_bounds__(kHistThreads)
k_hist(const uint64_t *__restrict__ keys, uint64_t n, const BatchCtrl *ctrl, uint32_t *hist) {
    __shared__ uint32_t sh[kMaxPasses * kRadix];
    if (ctrl->skip || !ctrl->run_sort) return;
    const SortPlan p = ctrl->plan;
    if (p.n_passes == 0) return;
    const DigitSel sel0 = digit_sel(p, 0);
    for (int i = threadIdx.x; i < kMaxPasses * kRadix; i += kHistThreads) sh[i] = 0u;
    __syncthreads();
    const uint64_t stride = (uint64_t)gridDim.x * kHistThreads;
    const uint64_t n_round = (n + 31ull) & ~31ull;         // whole warps stay in the loop together
    for (uint64_t i = (uint64_t)blockIdx.x * kHistThreads + threadIdx.x; i < n_round; i += stride) {
        const bool valid = i < n;
        const uint64_t ck = valid ? keys[i] : 0ull;
        for (uint32_t k = 0; k < 1u; ++k) {
            const uint32_t d = valid ? digit_at(ck, sel0) : 0xffffffffu;
            // the high digits of neighbouring keys are mostly equal, the low ones mostly all different: one vote tells the
            // two cases apart, and neither needs the lane-by-lane match (measured: 8.0 ms of a 58 ms sort at 200 M with it)
            const uint32_t d0 = __shfl_sync(0xffffffffu, d, 0);
            if (__all_sync(0xffffffffu, d == d0)) {
                if (lane_id() == 0 && valid) atomicAdd(&sh[k * kRadix + d], 32u);   // (a whole warp inside the batch: i < n for lane 0 means all)
            } else if (valid) {
                atomicAdd(&sh[k * kRadix + d], 1u);
            }
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < kRadix; i += kHistThreads)
        if (sh[i]) atomicAdd(&hist[i], sh[i]);
}

// =====================================================================================================
// one onesweep pass: stable partition of (key, index) by one digit, in a single sweep.  Tiles take
// their number from a counter (so every predecessor of a running tile has started), rank their keys
// per warp (equal digits are found through bit masks in shared memory), publish the tile's digit counts and look back over earlier tiles for the
// running totals.  Look-back words carry flag and count in one 32-bit word.
// =====================================================================================================
constexpr int kSortThreads = 512;
constexpr int kSortItems = 8;
constexpr int kSortTile = kSortThreads * kSortItems;     // 4096
constexpr int kSortWarps = kSortThreads / 32;
constexpr size_t kSortSmem = (size_t)kSortTile * 12 + (size_t)kSortWarps * kRadix * 4;
constexpr uint32_t kFlagAgg = 1u << 30, kFlagPrefix = 2u << 30, kCountMask = (1u << 30) - 1u;

// (three resident blocks per SM: at one block of 80 registers the pass ran at 13 % of the DRAM rate with a quarter of the
// warp slots in use, 4.1 ms for 200 M keys; bounded to 40 registers, with a few spills, it takes 2.5 ms)
__global__ void __launch_bounds__(kSortThreads, 3)
k_sort_pass(int pass, uint64_t n, BatchCtrl *ctrl, DevState *state, uint32_t *hist,
            uint64_t *keys0, uint64_t *keys1, uint32_t *idx0, uint32_t *idx1, uint32_t *desc0, uint32_t *desc1) {
    extern __shared__ __align__(16) unsigned char sort_smem[];
    uint64_t *s_keys = reinterpret_cast<uint64_t *>(sort_smem);                       // [kSortTile]
    uint32_t *s_idx = reinterpret_cast<uint32_t *>(s_keys + kSortTile);               // [kSortTile]
    uint32_t *s_cnt = s_idx + kSortTile;                                              // [kSortWarps][kRadix]
    __shared__ uint32_t s_local_start[kRadix];
    __shared__ uint32_t s_delta[kRadix];
    __shared__ uint32_t s_warp_tot[kRadix / 32], s_hist_tot[kRadix / 32];
    __shared__ uint32_t s_tile;
    __shared__ uint32_t s_next[kRadix];                     // this block's share of the next pass's histogram
    if (ctrl->skip || !ctrl->run_sort) return;
    const SortPlan &pl = ctrl->plan;
    if (pass >= (int)pl.n_passes) return;
    const bool count_next = pass + 1 < (int)pl.n_passes;
    const DigitSel sel = digit_sel(pl, pass), sel_next = digit_sel(pl, count_next ? pass + 1 : pass);
    if (threadIdx.x < kRadix) s_next[threadIdx.x] = 0u;
    const uint64_t *kin = (pass & 1) ? keys1 : keys0;
    uint64_t *kout = (pass & 1) ? keys0 : keys1;
    const uint32_t *iin = (pass & 1) ? idx1 : idx0;
    uint32_t *iout = (pass & 1) ? idx0 : idx1;
    uint32_t *desc = (pass & 1) ? desc1 : desc0;
    uint32_t *desc_next = (pass & 1) ? desc0 : desc1;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    const uint32_t n_tiles = (uint32_t)((n + kSortTile - 1) / kSortTile);
  for (;;) {                                  // persistent: tiles are taken in order from a counter
    __syncthreads();                          // shared memory of the previous tile is no longer read
    if (tid == 0) s_tile = atomicAdd(&ctrl->tile_counter[pass], 1u);
    for (int i = tid; i < kSortWarps * kRadix; i += kSortThreads) { s_cnt[i] = 0u; reinterpret_cast<uint32_t *>(s_keys)[i] = 0u; }
    __syncthreads();
    const uint32_t tile = s_tile;
    if (tile >= n_tiles) break;
    const uint32_t spin_limit = state->spin_limit;
    const bool mute = state->test_stage == 1u && pass == 0 && state->test_tile == tile;   // (test support: this tile stays silent)
    const uint64_t base = (uint64_t)tile * kSortTile;
    if (tid < kRadix) desc_next[(uint64_t)tile * kRadix + tid] = 0u;     // ready for the pass after this one

    const bool has_pad = base + kSortTile > n;                        // only the last tile holds padding
    // load, warp-striped: the warp's chunk is contiguous and item j of lane l sits at j*32 + l
    uint64_t key[kSortItems]; uint32_t rank[kSortItems];
    // (a key's digit is computed where it is needed: eight registers fewer than keeping it)
    auto digit_of = [&](uint64_t k) { return (has_pad && k == ~0ull) ? (uint32_t)(kRadix - 1) : digit_at(k, sel); };
    const uint64_t wbase = base + (uint64_t)warp * (32 * kSortItems);
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const uint64_t i = wbase + j * 32 + lane;
        key[j] = i < n ? kin[i] : ~0ull;                            // padding (no real key is all ones) ranks behind every real key
    }
    // the next pass's digit of every key, counted now (the high digits of neighbouring keys are mostly equal, the low ones
    // mostly all different: one vote over the warp's 256 keys tells the two cases apart)
    if (count_next) {
        auto next_digit = [&](int j) {
            return wbase + j * 32 + lane < n ? digit_at(key[j], sel_next) : 0xffffffffu;
        };
        // (equal digits: the keys agree on the digit's bits; a tile with padding takes the other branch)
        const uint64_t k0 = __shfl_sync(0xffffffffu, key[0], 0);
        uint64_t differ = has_pad ? ~0ull : 0ull;
#pragma unroll
        for (int j = 0; j < kSortItems; ++j) differ |= (key[j] ^ k0) & sel_next.raw;
        if (__all_sync(0xffffffffu, differ == 0ull)) {
            if (lane == 0) atomicAdd(&s_next[digit_at(k0, sel_next)], 32u * kSortItems);
        } else {
#pragma unroll
            for (int j = 0; j < kSortItems; ++j) {
                const uint32_t d2 = next_digit(j);
                if (d2 != 0xffffffffu) atomicAdd(&s_next[d2], 1u);
            }
        }
    }
    // rank inside the warp, in memory order.  Which lanes hold the same digit is found through shared memory: every lane
    // sets its bit in the digit's word of the warp's table (which lies where the tile's keys are put later) and reads the
    // word back; the highest of the lanes clears it and moves the warp's count on.  (`match_any` per key kept the unit that
    // executes it busier than any other: a pass took 2.4 ms at 200 M.)  A warp whose keys all share the digit needs no table.
    uint32_t *wcnt = s_cnt + warp * kRadix;
    uint32_t *wmask = reinterpret_cast<uint32_t *>(s_keys) + warp * kRadix;
    const uint64_t key0 = __shfl_sync(0xffffffffu, key[0], 0);
    uint64_t differ = has_pad ? ~0ull : 0ull;
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) differ |= (key[j] ^ key0) & sel.raw;
    const uint32_t dg0 = digit_at(key0, sel);
    if (__all_sync(0xffffffffu, differ == 0ull)) {           // all 256 keys of the warp: the high digits of input in order
#pragma unroll
        for (int j = 0; j < kSortItems; ++j) rank[j] = (uint32_t)(j * 32 + lane);
        if (lane == 0) wcnt[dg0] = 32u * kSortItems;
    } else {
#pragma unroll
        for (int j = 0; j < kSortItems; ++j) {
            const uint32_t dg = digit_of(key[j]);
            const uint32_t before = wcnt[dg];
            atomicOr(&wmask[dg], 1u << lane);
            __syncwarp();
            const unsigned peers = wmask[dg];
            rank[j] = before + (uint32_t)__popc(peers & lanemask_lt());
            __syncwarp();
            if ((peers >> lane) <= 1u) { wcnt[dg] = before + (uint32_t)__popc(peers); wmask[dg] = 0u; }    // highest peer lane writes
            __syncwarp();
        }
    }
    __syncthreads();

    // per digit: exclusive prefix over warps and the tile total; publish it; block-wide exclusive scans of
    // the tile's digit counts (positions inside the tile) and of the pass histogram (global digit starts)
    uint32_t tile_count = 0, local_incl = 0, hist_incl = 0, hist_mine = 0;
    if (tid < kRadix) {
#pragma unroll
        for (int w = 0; w < kSortWarps; ++w) { const uint32_t c = s_cnt[w * kRadix + tid]; s_cnt[w * kRadix + tid] = tile_count; tile_count += c; }
        if (!mute) st_relaxed_u32(desc + (uint64_t)tile * kRadix + tid, (tile == 0 ? kFlagPrefix : kFlagAgg) | tile_count);
        hist_mine = hist[pass * kRadix + tid];
        local_incl = tile_count; hist_incl = hist_mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, local_incl, o), u = __shfl_up_sync(0xffffffffu, hist_incl, o);
            if (lane >= o) { local_incl += t; hist_incl += u; }
        }
        if (lane == 31) { s_warp_tot[warp] = local_incl; s_hist_tot[warp] = hist_incl; }
    }
    __syncthreads();
    if (tid < kRadix) {
        uint32_t woff = 0, hoff = 0;
        for (int w = 0; w < warp; ++w) { woff += s_warp_tot[w]; hoff += s_hist_tot[w]; }
        const uint32_t local_start = local_incl - tile_count + woff;
        const uint32_t gstart = hist_incl - hist_mine + hoff;
        // look back over earlier tiles for the number of keys with this digit before this tile
        uint32_t excl = 0;
        bool failed = false;
        for (int64_t t = (int64_t)tile - 1; t >= 0; --t) {
            const uint32_t *p = desc + (uint64_t)t * kRadix + tid;
            uint32_t v = ld_relaxed_u32(p), spins = 0;
            while ((v >> 30) == 0u) {
                if (++spins > spin_limit) { failed = true; break; }
                __nanosleep(20);
                v = ld_relaxed_u32(p);
            }
            if (failed) break;
            excl += v & kCountMask;
            if ((v >> 30) == 2u) break;
        }
        // a wait that ran out: the batch is given up (later kernels of it exit at once) and the context is poisoned
        if (failed) { atomicExch(&ctrl->code, (int)HBF_E_TIMEOUT); ctrl->skip = 1; state->poisoned = 1; }
        if (tile != 0 && !mute) st_relaxed_u32(desc + (uint64_t)tile * kRadix + tid, kFlagPrefix | ((excl + tile_count) & kCountMask));
        s_local_start[tid] = local_start;
        s_delta[tid] = gstart + excl - local_start;
    }
    __syncthreads();

    // place keys at their position inside the tile, then write runs out (the indices are fetched only now: eight registers
    // fewer while the keys are ranked)
    uint32_t val[kSortItems];
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const uint64_t i = wbase + j * 32 + lane;
        val[j] = pass == 0 ? (uint32_t)i : (i < n ? iin[i] : 0u);
    }
#pragma unroll
    for (int j = 0; j < kSortItems; ++j) {
        const uint32_t dg = digit_of(key[j]);
        const uint32_t pos = s_local_start[dg] + wcnt[dg] + rank[j];
        s_keys[pos] = key[j]; s_idx[pos] = val[j];
    }
    __syncthreads();
    const int cnt = (int)min((uint64_t)kSortTile, n - base);
    for (int i = tid; i < cnt; i += kSortThreads) {
        const uint64_t k = s_keys[i];
        const uint32_t d = digit_at(k, sel);
        const uint32_t g = (uint32_t)i + s_delta[d];
        kout[g] = k; iout[g] = s_idx[i];
    }
  }
    // (the loop was left behind a block-wide barrier)
    if (count_next && tid < kRadix && s_next[tid]) atomicAdd(&hist[(pass + 1) * kRadix + tid], s_next[tid]);
}

// =====================================================================================================
// scan + scatter: in sorted order every access is the max-plus map B -> max(B + s, a + s); queues are
// segments.  A single-pass segmented scan with decoupled look-back gives each access the busy-until
// value it leaves behind; completion and stall go straight back to the access's own index, per-die
// totals are reduced with warp shuffles before they touch memory.
// =====================================================================================================
constexpr int kScanThreads = 256;
constexpr int kScanItems = 8;
constexpr int kScanTile = kScanThreads * kScanItems;     // 2048
constexpr int kScanWarps = kScanThreads / 32;

struct __align__(32) ScanDesc { int64_t S, M, value; uint32_t status; uint32_t pad; };
struct Map { int64_t S, M; int f; };

__device__ __forceinline__ Map compose(const Map &x, const Map &y) {      // x earlier, y later
    if (y.f) return y;
    Map r; r.f = x.f; r.S = x.S + y.S; r.M = max(x.M + y.S, y.M); return r;
}
__device__ __forceinline__ Map shfl_up_map(const Map &m, int o) {
    Map r; r.S = __shfl_up_sync(0xffffffffu, m.S, o); r.M = __shfl_up_sync(0xffffffffu, m.M, o);
    r.f = __shfl_up_sync(0xffffffffu, m.f, o); return r;
}

// (two blocks per SM; three or four, or 512 threads with four items each, were measured slower: the kernel is bound by its
// scattered accesses, not by latency)
__global__ void __launch_bounds__(kScanThreads, 2)
k_scan(const uint64_t *__restrict__ terms, uint64_t n,
       const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl, DevState *state,
       const uint64_t *keys0, const uint64_t *keys1, const uint32_t *idx0, const uint32_t *idx1,
       ScanDesc *desc, const int64_t *__restrict__ busy, int64_t *busy_stage, hbf_die_stats_t *stats_stage,
       int64_t *__restrict__ completion, int64_t *__restrict__ stall,
       const unsigned long long *claim_limit_p, uint32_t *die_claims) {
    __shared__ ModelParams mp;
    __shared__ uint32_t s_first_q[kScanThreads], s_last_q[kScanThreads];
    __shared__ Map s_warp_map[kScanWarps];
    __shared__ int64_t s_tile_in;
    __shared__ uint32_t s_tile;
    __shared__ long long s_die_acc[6];
    __shared__ long long s_res[3];
    if (ctrl->skip || !ctrl->run_sort) return;
    const uint64_t m = ctrl->n_ready;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kScanThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
  for (;;) {                                  // persistent: tiles are taken in order from a counter
    __syncthreads();
    if (tid == 0) s_tile = atomicAdd(&ctrl->tile_counter[kMaxPasses], 1u);
    if (tid < 6) s_die_acc[tid] = 0;
    if (tid < 3) s_res[tid] = tid == 2 ? INT64_MIN : 0;
    __syncthreads();
    const uint32_t tile = s_tile;
    const uint64_t base = (uint64_t)tile * kScanTile;
    if (base >= m) break;
    const uint32_t np = ctrl->plan.n_passes;
    const uint64_t *keys = (np & 1u) ? keys1 : keys0;
    const uint32_t *idxs = np == 0u ? nullptr : ((np & 1u) ? idx1 : idx0);
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const int cnt = (int)min((uint64_t)kScanTile, m - base);
    // retention on: a modeled access with a batch index below the claim limit pays one refresh quantum (a page read
    // and a page program, scaled like any service, Eq. 3) before its own service
    const uint64_t claim_limit = claim_limit_p ? *claim_limit_p : 0ull;
    const int64_t quantum_ns = q_ppm == 1000000 ? mp.t_read_ns + mp.t_prog_ns
        : (int64_t)div64((uint64_t)(mp.t_read_ns + mp.t_prog_ns) * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);

    // this thread's consecutive items
    uint32_t queue[kScanItems], idx[kScanItems], post[kScanItems];
    int64_t a[kScanItems], s[kScanItems], issue[kScanItems];
    const int t0 = tid * kScanItems;
    const int mine = max(0, min(kScanItems, cnt - t0));
    {
        uint64_t k[kScanItems];
        if (mine == kScanItems) {
            const ulonglong2 *k2 = reinterpret_cast<const ulonglong2 *>(keys + base + t0);
#pragma unroll
            for (int j = 0; j < kScanItems / 2; ++j) { const ulonglong2 v = k2[j]; k[2 * j] = v.x; k[2 * j + 1] = v.y; }
            if (idxs) {
                const uint4 *i4 = reinterpret_cast<const uint4 *>(idxs + base + t0);
#pragma unroll
                for (int j = 0; j < kScanItems / 4; ++j) { const uint4 v = i4[j]; idx[4 * j] = v.x; idx[4 * j + 1] = v.y; idx[4 * j + 2] = v.z; idx[4 * j + 3] = v.w; }
            } else {
#pragma unroll
                for (int j = 0; j < kScanItems; ++j) idx[j] = (uint32_t)(base + t0 + j);
            }
        } else {
#pragma unroll
            for (int j = 0; j < kScanItems; ++j) {
                k[j] = j < mine ? keys[base + t0 + j] : 0ull;
                idx[j] = j < mine ? (idxs ? idxs[base + t0 + j] : (uint32_t)(base + t0 + j)) : 0u;
            }
        }
#pragma unroll
        for (int j = 0; j < kScanItems; ++j) { queue[j] = (uint32_t)(k[j] >> kIssueBits); issue[j] = (int64_t)(k[j] & kIssueMask); }
    }
    // gather the records and rebuild their service terms
    long long acc_busy = 0, acc_br = 0, acc_bp = 0, acc_e = 0, acc_nr = 0, acc_np = 0;
    uint32_t acc_claims = 0;                                 // refresh quanta claimed on the die of the run in progress
    uint32_t run_die = 0xffffffffu;
    auto flush_run = [&](uint32_t die) {
        long long *d = reinterpret_cast<long long *>(stats_stage + die);
        if (acc_busy) atomicAdd((unsigned long long *)&d[0], (unsigned long long)acc_busy);
        if (acc_br) atomicAdd((unsigned long long *)&d[1], (unsigned long long)acc_br);
        if (acc_bp) atomicAdd((unsigned long long *)&d[2], (unsigned long long)acc_bp);
        if (acc_e) atomicAdd((unsigned long long *)&d[3], (unsigned long long)acc_e);
        if (acc_nr) atomicAdd((unsigned long long *)&d[4], (unsigned long long)acc_nr);
        if (acc_np) atomicAdd((unsigned long long *)&d[5], (unsigned long long)acc_np);
        if (acc_claims) atomicAdd(&die_claims[die], acc_claims);
        acc_busy = acc_br = acc_bp = acc_e = acc_nr = acc_np = 0; acc_claims = 0;
    };
    // what the scan needs of a record is the 8-byte word the classify kernel left for it (one 32-byte sector per access
    // instead of the 24-byte record, and no second classification or decode)
    uint64_t r_tw[kScanItems];
#pragma unroll
    for (int j = 0; j < kScanItems; ++j)
        if (j < mine) r_tw[j] = ld_nc_u64(terms + idx[j]);
    long long sum_s = 0;
#pragma unroll
    for (int j = 0; j < kScanItems; ++j) {
        if (j < mine) {
            const uint32_t bytes = (uint32_t)r_tw[j], op = (uint32_t)(r_tw[j] >> 32) & 1u, npages = (uint32_t)(r_tw[j] >> 33);
            const uint32_t die = mp.queue_level != 0u ? queue[j] : (mp.pow2_geom ? queue[j] >> mp.plane_shift : queue[j] / mp.planes);
            const Terms t = service_terms(mp, bytes, npages, op, q_ppm, div_q);
            s[j] = t.s;
            if (op) { a[j] = issue[j] + t.xfer; post[j] = 0u; } else { a[j] = issue[j]; post[j] = (uint32_t)t.xfer; }
            if (die != run_die) { if (run_die != 0xffffffffu) flush_run(run_die); run_die = die; }
            if ((uint64_t)idx[j] < claim_limit) { s[j] += quantum_ns; ++acc_claims; }
            acc_busy += s[j]; acc_e += t.energy; sum_s += s[j];
            if (op) { acc_bp += t.cb; acc_np += 1; } else { acc_br += t.cb; acc_nr += 1; }
        }
    }
    // segment heads: a queue change against the previous sorted element
    s_first_q[tid] = mine > 0 ? queue[0] : 0xffffffffu;
    s_last_q[tid] = mine > 0 ? queue[mine - 1] : 0xffffffffu;
    __syncthreads();
    uint32_t prev_q, next_q;
    if (tid > 0) prev_q = s_last_q[tid - 1];
    else prev_q = base > 0 ? (uint32_t)(keys[base - 1] >> kIssueBits) : 0xffffffffu;
    if (t0 + mine < cnt) next_q = s_first_q[tid + 1];
    else next_q = (base + cnt < m) ? (uint32_t)(keys[base + cnt] >> kIssueBits) : 0xffffffffu;

    // thread-local fold, then block scan of the thread maps
    Map tm; tm.f = 0; tm.S = 0; tm.M = kNegInf;
    {
        uint32_t pq = prev_q;
#pragma unroll
        for (int j = 0; j < kScanItems; ++j) {
            if (j < mine) {
                Map e; e.S = s[j]; e.f = queue[j] != pq;
                e.M = e.f ? max(busy[queue[j]], a[j]) + s[j] : a[j] + s[j];
                tm = compose(tm, e);
                pq = queue[j];
            }
        }
    }
    Map incl = tm;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const Map up = shfl_up_map(incl, o); if (lane >= o) incl = compose(up, incl); }
    if (lane == 31) s_warp_map[warp] = incl;
    __syncthreads();
    Map wprefix; wprefix.f = 0; wprefix.S = 0; wprefix.M = kNegInf;
    for (int w = 0; w < warp; ++w) wprefix = compose(wprefix, s_warp_map[w]);
    Map excl = shfl_up_map(incl, 1);
    if (lane == 0) { excl.f = 0; excl.S = 0; excl.M = kNegInf; }
    excl = compose(wprefix, excl);

    // tile aggregate, publish, look back
    if (tid == kScanThreads - 1) {
        const Map agg = compose(excl, tm);
        ScanDesc *my = desc + tile;
        int64_t tile_in = 0;
        const uint32_t spin_limit = state->spin_limit;
        const bool mute = state->test_stage == 2u && state->test_tile == tile;        // (test support: this tile stays silent)
        if (mute) {
        } else if (agg.f) {
            st_relaxed_s64(&my->value, agg.M);
            st_release_u32(&my->status, 2u);
            // the tile's own first segment may still continue the previous tile's queue
        } else {
            st_relaxed_s64(&my->S, agg.S); st_relaxed_s64(&my->M, agg.M);
            st_release_u32(&my->status, 1u);
        }
        // incoming busy-until for the tile's first element (unused when that element is a segment head)
        if (tile > 0) {
            int64_t S_acc = 0, M_acc = kNegInf;
            bool failed = false;
            for (int64_t t = (int64_t)tile - 1; t >= 0; --t) {
                const ScanDesc *p = desc + t;
                uint32_t stt = ld_acquire_u32(&p->status), spins = 0;
                while (stt == 0u) {
                    if (++spins > spin_limit) { failed = true; break; }
                    __nanosleep(20);
                    stt = ld_acquire_u32(&p->status);
                }
                if (failed) break;
                if (stt == 2u) {
                    // a later upgrade from 1 to 2 is also fine: value is complete once status reads 2
                    const int64_t v = ld_relaxed_s64(&p->value);
                    tile_in = max(v + S_acc, M_acc);
                    break;
                }
                const int64_t St = ld_relaxed_s64(&p->S), Mt = ld_relaxed_s64(&p->M);
                M_acc = max(Mt + S_acc, M_acc); S_acc += St;
            }
            if (failed) { atomicExch(&ctrl->code, (int)HBF_E_TIMEOUT); ctrl->skip = 1; state->poisoned = 1; }
        }
        if (!agg.f && !mute) {
            st_relaxed_s64(&my->value, max(tile_in + agg.S, agg.M));
            st_release_u32(&my->status, 2u);
        }
        s_tile_in = tile_in;
    }
    __syncthreads();
    int64_t B = excl.f ? excl.M : max(s_tile_in + excl.S, excl.M);

    // apply: serve this thread's items in order
    long long sum_stall = 0, max_c = INT64_MIN;
    {
        uint32_t pq = prev_q;
#pragma unroll
        for (int j = 0; j < kScanItems; ++j) {
            if (j < mine) {
                if (queue[j] != pq) B = busy[queue[j]];
                const int64_t start = max(a[j], B);
                B = start + s[j];
                const int64_t c = B + (int64_t)post[j];
                completion[idx[j]] = c;                      // (the stalls follow from a sequential pass: half the scattered writes)
                sum_stall += c - issue[j];
                max_c = max(max_c, (long long)c);
                const uint32_t nq = j + 1 < mine ? queue[j + 1] : next_q;
                if (nq != queue[j]) busy_stage[queue[j]] = B;       // last access of its queue in this batch
                pq = queue[j];
            }
        }
    }
    // per-die totals: whole warps on one die reduce by shuffle into the tile's slot
    {
        const uint32_t tile_die = __shfl_sync(0xffffffffu, run_die, 0);
        const bool uniform = __all_sync(0xffffffffu, run_die == tile_die || run_die == 0xffffffffu) && tile_die != 0xffffffffu;
        __shared__ uint32_t s_tile_die;
        if (tid == 0) s_tile_die = run_die;
        __syncthreads();
        if (uniform && tile_die == s_tile_die) {
            acc_busy = warp_sum(acc_busy); acc_br = warp_sum(acc_br); acc_bp = warp_sum(acc_bp);
            acc_e = warp_sum(acc_e); acc_nr = warp_sum(acc_nr); acc_np = warp_sum(acc_np);
            acc_claims = (uint32_t)warp_sum((long long)acc_claims);
            if (lane == 0 && acc_claims) atomicAdd(&die_claims[tile_die], acc_claims);
            if (lane == 0) {
                atomicAdd((unsigned long long *)&s_die_acc[0], (unsigned long long)acc_busy);
                atomicAdd((unsigned long long *)&s_die_acc[1], (unsigned long long)acc_br);
                atomicAdd((unsigned long long *)&s_die_acc[2], (unsigned long long)acc_bp);
                atomicAdd((unsigned long long *)&s_die_acc[3], (unsigned long long)acc_e);
                atomicAdd((unsigned long long *)&s_die_acc[4], (unsigned long long)acc_nr);
                atomicAdd((unsigned long long *)&s_die_acc[5], (unsigned long long)acc_np);
            }
        } else if (run_die != 0xffffffffu) {
            flush_run(run_die);
        }
        sum_stall = warp_sum(sum_stall); sum_s = warp_sum(sum_s); max_c = warp_max(max_c);
        if (lane == 0) {
            atomicAdd((unsigned long long *)&s_res[0], (unsigned long long)sum_stall);
            atomicAdd((unsigned long long *)&s_res[1], (unsigned long long)sum_s);
            atomicMax(&s_res[2], max_c);
        }
        __syncthreads();
        if (tid == 0) {
            long long *d = reinterpret_cast<long long *>(stats_stage + s_tile_die);
            for (int k = 0; k < 6; ++k) if (s_die_acc[k]) atomicAdd((unsigned long long *)&d[k], (unsigned long long)s_die_acc[k]);
            atomicAdd((unsigned long long *)&ctrl->modeled_ns, (unsigned long long)s_res[0]);
            atomicAdd((unsigned long long *)&ctrl->service_ns, (unsigned long long)s_res[1]);
            atomicMax(&ctrl->max_completion_ns, s_res[2]);
        }
    }
  }
}

// stalls of a batch the sort path served: stall = completion - issue, in batch order (coalesced reads and writes; the scan
// scatters completions only).  Rows that are not modeled have completion = issue, hence no stall.
__global__ void __launch_bounds__(256)
k_stalls(const hbf_access_t *__restrict__ acc, uint64_t n, const BatchCtrl *ctrl, const int64_t *__restrict__ completion,
         int64_t *__restrict__ stall) {
    if (ctrl->skip || !ctrl->run_sort) return;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x)
        stall[i] = completion[i] - (int64_t)__ldg(reinterpret_cast<const uint64_t *>(acc + i) + 1);
}

// =====================================================================================================
// finish: commit the staged state, or zero the outputs of a refused batch; write the batch summary
// =====================================================================================================
__global__ void k_finish(uint64_t n, BatchCtrl *ctrl, DevState *state, int64_t *busy, const int64_t *busy_stage,
                         int64_t *pending, const hbf_die_stats_t *stats_stage, hbf_die_stats_t *die_stats,
                         int64_t *completion, int64_t *stall, hbf_batch_result_t *result,
                         const ModelParams *__restrict__ mp, uint32_t n_queues, uint32_t n_dies, int binned, int bus_on) {
    int code = ctrl->code;
    // With the channel-bus stage on, array-done times become sort keys of 47 bits: a batch that reaches 2^47 ns is refused
    // here, before anything is committed (every array-done time is at most the largest completion).  Every thread reads
    // the same settled values, so every thread takes the same decision.
    if (bus_on && code == HBF_OK && ctrl->n_ready && ctrl->max_completion_ns >= HBF_ISSUE_LIMIT) code = HBF_E_INVAL;
    const uint64_t gtid = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (code == HBF_E_TIMEOUT && gtid == 0) state->poisoned = 1;         // a bounded device-side wait expired
    const uint64_t gsz = (uint64_t)gridDim.x * blockDim.x;
    if (code == HBF_E_ACCESS_FAULT || code == HBF_E_TIMEOUT || code == HBF_E_INVAL) {
        for (uint64_t i = gtid; i < n; i += gsz) { completion[i] = 0; stall[i] = 0; }
        if (die_stats) for (uint64_t i = gtid; i < (uint64_t)n_dies * 6u; i += gsz) reinterpret_cast<int64_t *>(die_stats)[i] = 0;
    } else if (code == HBF_OK) {
        const bool inorder = ctrl->inorder_used != 0u;
        for (uint64_t r = gtid; r < n_queues; r += gsz) busy[r] = busy_stage[r];
        for (uint64_t d = gtid; d < n_dies; d += gsz) {
            hbf_die_stats_t ds = stats_stage[d];
            // the in-order path keeps byte and access counts only: the energy is linear in them
            if (inorder) ds.energy_pj = mp->e_cmd_read_pj * ds.n_read + mp->e_byte_read_pj * ds.bytes_read +
                                        mp->e_cmd_prog_pj * ds.n_prog + mp->e_byte_prog_pj * ds.bytes_prog;
            if (!binned) pending[d] += ds.energy_pj;          // with the time-bin ledger on, the energy is booked per event
            if (die_stats) die_stats[d] = ds;
        }
    }
    if (gtid == 0) {
        hbf_batch_result_t r;
        r.code = code; r.mode = ctrl->mode; r.q_ppm = ctrl->q_ppm;
        r.n_native = code == HBF_OK || code == HBF_E_ACCESS_FAULT ? ctrl->n_native : 0;
        r.n_modeled = code == HBF_OK ? ctrl->n_ready : 0;
        r.n_fault = ctrl->n_fault;
        r.modeled_ns = code == HBF_OK ? ctrl->modeled_ns : 0;
        r.service_ns = code == HBF_OK ? ctrl->service_ns : 0;
        r.max_completion_ns = code == HBF_OK && ctrl->n_ready ? ctrl->max_completion_ns : 0;
        *result = r;
    }
}

// copy of the served order out of the workspace (sort path only)
__global__ void k_queue_order(const BatchCtrl *ctrl, const uint32_t *idx0, const uint32_t *idx1, uint32_t *out, uint64_t n) {
    const uint64_t m = ctrl->n_ready;
    const uint32_t np = ctrl->plan.n_passes;
    const uint32_t *src = np == 0u ? nullptr : ((np & 1u) ? idx1 : idx0);
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < m && i < n; i += (uint64_t)gridDim.x * blockDim.x)
        out[i] = src ? src[i] : (uint32_t)i;
}

// =====================================================================================================
// channel bus as a second queued stage (an extension; the library's own definition).  After the array
// stage, a read's data-out transfer queues on the bus of its channel in (array-done time, index) order and
// holds it for the transfer time; the read completes when the transfer does.  Programs are unchanged.
//   keys   per access: channel << 47 | array-done time (reads), a sentinel behind every channel (the rest)
//   sort   the onesweep passes of the sort path, over the key bits that differ
//   scan   in sorted order a read is the map B -> max(B, D) + x on its channel's bus; channels are segments
//          whose first map starts from the bus state earlier batches left.  Three kernels, no look-back: tile
//          aggregates, an exclusive scan of them by one block, tiles again with their carry.
// =====================================================================================================
struct BusMap { int64_t S, M; int f; };                    // B -> max(B + S, M); f: contains a segment head (then B does not matter)
__device__ __forceinline__ BusMap bus_then(const BusMap &a, const BusMap &b) {       // a first, then b
    if (b.f) return b;
    BusMap r; r.S = a.S + b.S; r.M = max((int64_t)(a.M + b.S), b.M); r.f = a.f; return r;
}
__device__ __forceinline__ BusMap bus_identity() { BusMap r; r.S = 0; r.M = kNegInf; r.f = 0; return r; }
__device__ __forceinline__ BusMap bus_shfl_up(const BusMap &v, int o) {
    BusMap r; r.S = __shfl_up_sync(0xffffffffu, v.S, o); r.M = __shfl_up_sync(0xffffffffu, v.M, o); r.f = __shfl_up_sync(0xffffffffu, v.f, o);
    return r;
}
constexpr int kBusThreads = 256;
constexpr int kBusItems = 8;
constexpr int kBusTile = kBusThreads * kBusItems;          // as many entries as a scan tile of the sort path: its descriptors are reused
static_assert(kBusTile == kScanTile && sizeof(BusMap) <= sizeof(ScanDesc), "the bus stage reuses the scan descriptors");

__global__ void k_bus_begin(BatchCtrl *bc, const hbf_batch_result_t *result, uint32_t *hist) {
    uint32_t *w = reinterpret_cast<uint32_t *>(bc);
    for (int i = threadIdx.x; i < (int)(sizeof(BatchCtrl) / 4); i += blockDim.x) w[i] = 0u;
    for (int i = threadIdx.x; i < kMaxPasses * kRadix; i += blockDim.x) hist[i] = 0u;
    __syncthreads();
    if (threadIdx.x == 0) {
        bc->key_and = ~0ull; bc->run_sort = 1u; bc->unsorted = 1u;
        bc->max_completion_ns = INT64_MIN;
        if (result->code != HBF_OK) bc->skip = 1;           // a refused batch has no second stage
    }
}

__global__ void __launch_bounds__(256)
k_bus_keys(const hbf_access_t *__restrict__ acc, uint64_t n, const int64_t *__restrict__ completion,
           const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp_g, BatchCtrl *bc,
           uint64_t *__restrict__ keys, uint32_t *__restrict__ xfer_out) {
    __shared__ ModelParams mp;
    if (bc->skip) return;
    for (int i = threadIdx.x; i < (int)(sizeof(ModelParams) / 4); i += blockDim.x)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    __syncthreads();
    const RangeSnap &rs = *ranges;
    const uint64_t sentinel = (uint64_t)mp.channels << kIssueBits;
    const Div64 one = make_div64(1000000ull);
    unsigned long long reads = 0, k_or = 0, k_and = ~0ull;
    unsigned late = 0;
    const uint64_t n_round = (n + 31ull) & ~31ull;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_round; i += (uint64_t)gridDim.x * blockDim.x) {
        if (i >= n) continue;
        const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
        const uint64_t addr = __ldg(rec), bf = __ldg(rec + 2);
        const int64_t issue = (int64_t)__ldg(rec + 1);
        const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
        int g = 0;
        uint64_t key = sentinel;
        uint32_t x = 0;
        if (classify(rs, addr, issue, bytes, flags, &g) == HBF_ST_READY && !(flags & 1u)) {
            const Decoded d = decode(mp, rs.media_offset[g] + (addr - rs.base[g]), bytes);
            const Terms t = service_terms(mp, bytes, d.npages, 0u, 1000000, one);      // the transfer does not depend on the throttle
            const int64_t done = completion[i] - t.xfer;                                 // when the array is done with the read
            x = (uint32_t)t.xfer;
            if (done < 0 || done >= HBF_ISSUE_LIMIT) late = 1u;
            else { key = ((uint64_t)(d.die / mp.dies) << kIssueBits) | (uint64_t)done; ++reads; }
        }
        keys[i] = key; xfer_out[i] = x;
        k_or |= key; k_and &= key;
    }
    reads = (unsigned long long)warp_sum((long long)reads);
    k_or = warp_or(k_or); k_and = warp_and(k_and);
    late = __any_sync(0xffffffffu, late);
    if (lane_id() == 0) {
        if (reads) atomicAdd(&bc->n_ready, reads);
        atomicOr(&bc->key_or, k_or); atomicAnd(&bc->key_and, k_and);
        if (late) atomicExch(&bc->code, (int)HBF_E_INVAL);  // an array-done time beyond the 47-bit key field
    }
}

__global__ void k_bus_check(BatchCtrl *bc) { if (bc->code != HBF_OK) bc->skip = 1; }

// entry j of the sorted order as a map on its channel's bus
__device__ __forceinline__ BusMap bus_entry(uint64_t j, const uint64_t *__restrict__ ks, const uint32_t *__restrict__ is, bool have_idx,
                                            const uint32_t *__restrict__ xfer, const uint32_t *xs, const int64_t *__restrict__ bus_busy,
                                            uint32_t *idx_out, uint32_t *ch_out, int64_t *plain_out, uint32_t *x_out) {
    const uint64_t key = ks[j];
    const uint32_t ch = (uint32_t)(key >> kIssueBits), idx = have_idx ? is[j] : (uint32_t)j;
    // the transfer time: by batch index from the array the keys kernel wrote (a gather), or in sorted order from the copy the
    // reduce pass made of what it gathered
    const uint32_t xr = xs ? xs[j] : xfer[idx];
    *x_out = xr;
    const int64_t done = (int64_t)(key & kIssueMask), x = (int64_t)xr;
    const bool head = j == 0 || (uint32_t)(ks[j - 1] >> kIssueBits) != ch;
    BusMap m; m.S = x; m.M = (head ? max(bus_busy[ch], done) : done) + x; m.f = head ? 1 : 0;
    *idx_out = idx; *ch_out = ch; *plain_out = done + x;
    return m;
}

__global__ void __launch_bounds__(kBusThreads)
k_bus_reduce(const BatchCtrl *bc, const uint64_t *k0, const uint64_t *k1, uint32_t *i0, uint32_t *i1,
             const uint32_t *__restrict__ xfer, const int64_t *__restrict__ bus_busy, ScanDesc *agg) {
    __shared__ BusMap s_warp[kBusThreads / 32];
    if (bc->skip) return;
    const uint64_t m = bc->n_ready;
    const uint32_t np = bc->plan.n_passes;
    const uint64_t *ks = (np & 1u) ? k1 : k0; const uint32_t *is = (np & 1u) ? i1 : i0;
    uint32_t *xs = np != 0u ? ((np & 1u) ? i0 : i1) : nullptr;      // the index buffer the sort no longer needs (no passes: the order is the batch's)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (uint64_t tile = blockIdx.x; tile * kBusTile < m; tile += gridDim.x) {
        BusMap mine = bus_identity();
        const uint64_t first = tile * kBusTile + (uint64_t)tid * kBusItems;
        for (int u = 0; u < kBusItems; ++u) {
            const uint64_t j = first + u;
            if (j >= m) break;
            uint32_t idx, ch, x; int64_t plain;
            mine = bus_then(mine, bus_entry(j, ks, is, np != 0u, xfer, nullptr, bus_busy, &idx, &ch, &plain, &x));
            if (xs) xs[j] = x;                               // for the apply pass: it reads this in order instead of gathering again
        }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const BusMap p = bus_shfl_up(mine, o); if (lane >= o) mine = bus_then(p, mine); }
        __syncthreads();
        if (lane == 31) s_warp[warp] = mine;
        __syncthreads();
        if (tid == 0) {
            BusMap t = s_warp[0];
            for (int w = 1; w < kBusThreads / 32; ++w) t = bus_then(t, s_warp[w]);
            ScanDesc d; d.S = t.S; d.M = t.M; d.value = 0; d.status = (uint32_t)t.f; d.pad = 0;
            agg[tile] = d;
        }
    }
}

// one block: exclusive scan (in tile order) of the tile aggregates, in place
__global__ void __launch_bounds__(1024)
k_bus_tile_scan(const BatchCtrl *bc, ScanDesc *agg) {
    __shared__ BusMap s_warp[32];
    if (bc->skip) return;
    const uint64_t tiles = (bc->n_ready + kBusTile - 1) / kBusTile;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint64_t per = (tiles + 1023) / 1024, lo = (uint64_t)tid * per, hi = min(tiles, lo + per);
    BusMap mine = bus_identity();
    for (uint64_t t = lo; t < hi; ++t) { BusMap e; e.S = agg[t].S; e.M = agg[t].M; e.f = (int)agg[t].status; mine = bus_then(mine, e); }
    BusMap incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const BusMap p = bus_shfl_up(incl, o); if (lane >= o) incl = bus_then(p, incl); }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    BusMap before = bus_identity();
    for (int w = 0; w < warp; ++w) before = bus_then(before, s_warp[w]);
    BusMap prev = bus_shfl_up(incl, 1);
    if (lane == 0) prev = bus_identity();
    BusMap run = bus_then(before, prev);                    // everything before this thread's tiles
    for (uint64_t t = lo; t < hi; ++t) {
        BusMap e; e.S = agg[t].S; e.M = agg[t].M; e.f = (int)agg[t].status;
        ScanDesc d; d.S = run.S; d.M = run.M; d.value = 0; d.status = (uint32_t)run.f; d.pad = 0;
        agg[t] = d;
        run = bus_then(run, e);
    }
}

__global__ void __launch_bounds__(kBusThreads)
k_bus_apply(const hbf_access_t *__restrict__ acc, BatchCtrl *bc, const uint64_t *k0, const uint64_t *k1, const uint32_t *i0,
            const uint32_t *i1, const uint32_t *__restrict__ xfer, int64_t *bus_busy, const ScanDesc *__restrict__ agg,
            int64_t *__restrict__ completion, int64_t *__restrict__ stall) {
    __shared__ BusMap s_warp[kBusThreads / 32];
    if (bc->skip) return;
    const uint64_t m = bc->n_ready;
    const uint32_t np = bc->plan.n_passes;
    const uint64_t *ks = (np & 1u) ? k1 : k0; const uint32_t *is = (np & 1u) ? i1 : i0;
    const uint32_t *xs = np != 0u ? ((np & 1u) ? i0 : i1) : nullptr;    // the transfer times in sorted order, left by the reduce pass
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    long long moved = 0, max_c = INT64_MIN;
    for (uint64_t tile = blockIdx.x; tile * kBusTile < m; tile += gridDim.x) {
        const uint64_t first = tile * kBusTile + (uint64_t)tid * kBusItems;
        BusMap e[kBusItems]; uint32_t idx[kBusItems], ch[kBusItems]; int64_t plain[kBusItems];
        BusMap mine = bus_identity();
#pragma unroll
        for (int u = 0; u < kBusItems; ++u) {
            const uint64_t j = first + u;
            uint32_t x;
            if (j < m) { e[u] = bus_entry(j, ks, is, np != 0u, xfer, xs, bus_busy, &idx[u], &ch[u], &plain[u], &x); mine = bus_then(mine, e[u]); }
            else { e[u] = bus_identity(); idx[u] = 0; ch[u] = 0; plain[u] = 0; }
        }
        BusMap incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const BusMap p = bus_shfl_up(incl, o); if (lane >= o) incl = bus_then(p, incl); }
        __syncthreads();
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        BusMap run; run.S = agg[tile].S; run.M = agg[tile].M; run.f = (int)agg[tile].status;     // everything before the tile
        for (int w = 0; w < warp; ++w) run = bus_then(run, s_warp[w]);
        BusMap prev = bus_shfl_up(incl, 1);
        if (lane == 0) prev = bus_identity();
        run = bus_then(run, prev);
        // Every prefix holds a segment head (entry 0 is one), so the composed map's constant term is the bus's
        // busy-until after the entry: the time the read's transfer ends.
#pragma unroll
        for (int u = 0; u < kBusItems; ++u) {
            const uint64_t j = first + u;
            if (j >= m) break;
            run = bus_then(run, e[u]);
            const int64_t done = run.M;
            if (done != plain[u]) {                          // the transfer waited for the bus: completion and stall move by the wait
                completion[idx[u]] = done; stall[idx[u]] += done - plain[u];
                moved += done - plain[u]; max_c = max(max_c, (long long)done);
            }
        }
    }
    moved = warp_sum(moved); max_c = warp_max(max_c);
    if (lane == 0) {
        if (moved) atomicAdd((unsigned long long *)&bc->modeled_ns, (unsigned long long)moved);
        if (max_c != INT64_MIN) atomicMax(&bc->max_completion_ns, max_c);
    }
}

// The bus state is written by a pass of its own, after every tile has read the old one: the last read of each
// channel's segment holds the new busy-until in its completion.
__global__ void __launch_bounds__(256)
k_bus_commit(const BatchCtrl *bc, const uint64_t *k0, const uint64_t *k1, const uint32_t *i0, const uint32_t *i1,
             const int64_t *__restrict__ completion, int64_t *bus_busy) {
    if (bc->skip) return;
    const uint64_t m = bc->n_ready;
    const uint32_t np = bc->plan.n_passes;
    const uint64_t *ks = (np & 1u) ? k1 : k0; const uint32_t *is = (np & 1u) ? i1 : i0;
    for (uint64_t j = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; j < m; j += (uint64_t)gridDim.x * blockDim.x) {
        const uint32_t ch = (uint32_t)(ks[j] >> kIssueBits);
        if (j + 1 == m || (uint32_t)(ks[j + 1] >> kIssueBits) != ch) bus_busy[ch] = completion[np ? is[j] : (uint32_t)j];
    }
}

__global__ void k_bus_finish(const BatchCtrl *bc, hbf_batch_result_t *result, DevState *state) {
    if (bc->code != HBF_OK) { result->code = bc->code; state->poisoned = 1; return; }   // the array stage is committed: the context cannot go on
    if (bc->skip) return;
    result->modeled_ns += bc->modeled_ns;
    if (bc->max_completion_ns > result->max_completion_ns) result->max_completion_ns = bc->max_completion_ns;
}

cudaError_t launch_bus_stage(const SubmitArgs &a, BatchCtrl *bc, int64_t *bus_busy, cudaStream_t st) {
    const uint64_t n = a.n;
    if (n == 0) return cudaSuccess;
    const uint64_t sort_tiles = (n + kSortTile - 1) / kSortTile, bus_tiles = (n + kBusTile - 1) / kBusTile;
    cudaError_t e = cudaMemsetAsync(a.ws.sort_desc[0], 0, sort_tiles * kRadix * 4, st);
    if (e != cudaSuccess) return e;
    k_bus_begin<<<1, 256, 0, st>>>(bc, a.result, a.ws.hist);
    const unsigned wide = (unsigned)std::min<uint64_t>((n + 255) / 256, (uint64_t)a.sm_count * 8);
    k_bus_keys<<<wide, 256, 0, st>>>(a.acc, n, a.completion, a.ranges, a.mp_dev, bc, a.ws.keys[0], a.ws.bus_xfer);
    k_bus_check<<<1, 1, 0, st>>>(bc);
    k_plan<<<1, 32, 0, st>>>(bc, 1);
    const unsigned hist_grid = (unsigned)std::min<uint64_t>((n + kHistThreads * 8 - 1) / (kHistThreads * 8), (uint64_t)a.sm_count * 4);
    k_hist<<<hist_grid, kHistThreads, 0, st>>>(a.ws.keys[0], n, bc, a.ws.hist);
    e = ensure_dyn_smem((const void *)k_sort_pass, kSortSmem);
    if (e != cudaSuccess) return e;
    const unsigned sort_grid = (unsigned)std::min<uint64_t>(sort_tiles, (uint64_t)a.sm_count * 3);
    for (int p = 0; p < kMaxPasses; ++p)
        k_sort_pass<<<sort_grid, kSortThreads, kSortSmem, st>>>(p, n, bc, a.state, a.ws.hist, a.ws.keys[0], a.ws.keys[1],
                                                                a.ws.idx[0], a.ws.idx[1], a.ws.sort_desc[0], a.ws.sort_desc[1]);
    k_bus_check<<<1, 1, 0, st>>>(bc);                        // a look-back that gave up sets the code
    const unsigned tiles_grid = (unsigned)std::min<uint64_t>(bus_tiles, (uint64_t)a.sm_count * 8);
    ScanDesc *agg = (ScanDesc *)a.ws.scan_desc;
    k_bus_reduce<<<tiles_grid, kBusThreads, 0, st>>>(bc, a.ws.keys[0], a.ws.keys[1], a.ws.idx[0], a.ws.idx[1], a.ws.bus_xfer, bus_busy, agg);
    k_bus_tile_scan<<<1, 1024, 0, st>>>(bc, agg);
    k_bus_apply<<<tiles_grid, kBusThreads, 0, st>>>(a.acc, bc, a.ws.keys[0], a.ws.keys[1], a.ws.idx[0], a.ws.idx[1], a.ws.bus_xfer, bus_busy,
                                                    agg, a.completion, a.stall);
    k_bus_commit<<<wide, 256, 0, st>>>(bc, a.ws.keys[0], a.ws.keys[1], a.ws.idx[0], a.ws.idx[1], a.completion, bus_busy);
    k_bus_finish<<<1, 1, 0, st>>>(bc, a.result, a.state);
    g_kernel_launches += 10 + kMaxPasses;
    return cudaGetLastError();
}

// =====================================================================================================
// host side
// =====================================================================================================
static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t workspace_layout(uint64_t n, uint32_t n_queues, Workspace *ws, void *base_ptr, int with_bus) {
    const uint64_t nn = n ? n : 1;
    const uint64_t sort_tiles = (nn + kSortTile - 1) / kSortTile, scan_tiles = (nn + kScanTile - 1) / kScanTile;
    size_t off = 0;
    char *b = static_cast<char *>(base_ptr);
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return b ? b + o : nullptr; };
    void *k0 = take(nn * 8), *k1 = take(nn * 8), *i0 = take(nn * 4), *i1 = take(nn * 4);
    void *tw = take(nn * 8);
    void *h = take((size_t)kMaxPasses * kRadix * 4);
    void *d0 = take(sort_tiles * kRadix * 4), *d1 = take(sort_tiles * kRadix * 4);
    void *sd = take(scan_tiles * sizeof(ScanDesc));
    const uint64_t in_tiles = inorder_tiles_bound(nn);
    const bool inorder = n_queues <= kInMaxQueues;
    void *ia = take(inorder ? in_tiles * n_queues * 16 : 0), *ib = take(inorder ? in_tiles * n_queues * 8 : 0);
    // (the tile table also takes one entry per block of the small-batch route, which a batch of few records has more of than tiles)
    void *it = take(inorder ? std::max<uint64_t>(in_tiles, inorder_small_blocks(n_queues)) * sizeof(InTile) : 0);
    void *ih = take(inorder ? inorder_head_bytes(in_tiles, n_queues) : 0);
    void *ic = take(inorder ? in_tiles * n_queues : 0);
    void *iq = take(inorder ? inorder_qid_entries(nn) * 2 : 0);
    void *bx = take(with_bus ? nn * 4 : 0);
    if (ws) {
        ws->keys[0] = (uint64_t *)k0; ws->keys[1] = (uint64_t *)k1; ws->idx[0] = (uint32_t *)i0; ws->idx[1] = (uint32_t *)i1;
        ws->terms = (uint64_t *)tw;
        ws->hist = (uint32_t *)h; ws->sort_desc[0] = (uint32_t *)d0; ws->sort_desc[1] = (uint32_t *)d1;
        ws->scan_desc = sd; ws->in_agg = (int64_t *)ia; ws->in_bin = (int64_t *)ib;
        ws->in_tile = it; ws->in_head = ih; ws->in_headcnt = (uint8_t *)ic; ws->in_qid = (uint16_t *)iq; ws->bus_xfer = (uint32_t *)bx; ws->bytes = off;
    }
    return off;
}

std::atomic<unsigned long long> g_kernel_launches{0};

cudaError_t ensure_dyn_smem(const void *kernel, size_t bytes) {
    struct Entry { int device; const void *kernel; size_t bytes; };
    static std::mutex mu;
    static std::vector<Entry> set;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    for (Entry &en : set)
        if (en.device == dev && en.kernel == kernel) {
            if (bytes <= en.bytes) return cudaSuccess;
            e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
            if (e == cudaSuccess) en.bytes = bytes;
            return e;
        }
    if (bytes > 48u * 1024u) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e == cudaSuccess) set.push_back(Entry{dev, kernel, bytes});
    return e;
}

static cudaError_t launch_sort_path(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    auto mark = [&](int k) { if (a.ev) cudaEventRecord(a.ev[k], st); };
    const uint64_t sort_tiles = (n + kSortTile - 1) / kSortTile, scan_tiles = (n + kScanTile - 1) / kScanTile;
    cudaError_t e = cudaMemsetAsync(a.ws.sort_desc[0], 0, sort_tiles * kRadix * 4, st);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(a.ws.scan_desc, 0, scan_tiles * sizeof(ScanDesc), st);
    if (e != cudaSuccess) return e;
    mark(1);
    const uint64_t cls_tiles = (n + kClsTile - 1) / kClsTile;
    const unsigned cls_grid = (unsigned)std::min<uint64_t>(cls_tiles, (uint64_t)a.sm_count * 8);
    k_classify<<<cls_grid, kClsThreads, 0, st>>>(a.acc, n, a.ranges, a.mp_dev, a.ctrl, a.ws.keys[0], a.ws.terms, a.status,
                                                 a.completion, a.stall);
    mark(2);
    k_plan<<<1, 32, 0, st>>>(a.ctrl, a.path == HBF_PATH_SORT_FULL ? 1 : 0);
    const unsigned hist_grid = (unsigned)std::min<uint64_t>((n + kHistThreads * 8 - 1) / (kHistThreads * 8), (uint64_t)a.sm_count * 4);
    k_hist<<<hist_grid, kHistThreads, 0, st>>>(a.ws.keys[0], n, a.ctrl, a.ws.hist);
    mark(3);
    e = ensure_dyn_smem((const void *)k_sort_pass, kSortSmem);
    if (e != cudaSuccess) return e;
    const unsigned sort_grid = (unsigned)std::min<uint64_t>(sort_tiles, (uint64_t)a.sm_count * 3);
    for (int p = 0; p < kMaxPasses; ++p)
        k_sort_pass<<<sort_grid, kSortThreads, kSortSmem, st>>>(p, n, a.ctrl, a.state, a.ws.hist, a.ws.keys[0], a.ws.keys[1],
                                                                           a.ws.idx[0], a.ws.idx[1], a.ws.sort_desc[0], a.ws.sort_desc[1]);
    mark(4);
    k_scan<<<(unsigned)std::min<uint64_t>(scan_tiles, (uint64_t)a.sm_count * 8), kScanThreads, 0, st>>>(a.ws.terms, n, a.mp_dev, a.ctrl, a.state, a.ws.keys[0], a.ws.keys[1],
                                                         a.ws.idx[0], a.ws.idx[1], (ScanDesc *)a.ws.scan_desc, a.busy,
                                                         a.busy_stage, a.stats_stage, a.completion, a.stall,
                                                         a.claim_limit, a.die_claims);
    k_stalls<<<(unsigned)std::min<uint64_t>((n + 255) / 256, (uint64_t)a.sm_count * 16), 256, 0, st>>>(a.acc, n, a.ctrl, a.completion, a.stall);
    g_kernel_launches += 5 + kMaxPasses;
    return cudaSuccess;
}

// ---- the sort path launched from the device -----------------------------------------------------------
// With HBF_PATH_AUTO the host enqueues the in-order kernels only.  A batch that turns out not to be in issue
// order (or has a service time the in-order kernels cannot hold) needs the sort path after all, and the host
// cannot know that without waiting for the device.  So the kernel that follows the in-order kernels (it also sums the
// batch's stall total when they did serve it) looks at the batch's control block and, in that case only, one thread launches the sort path's kernels itself, in order, into the tail-launch stream: they run
// after this kernel and before the next kernel of the host's stream (a parent grid is complete
// only when its children are), which is the batch's finish kernel.  A batch in issue order pays one empty
// launch instead of thirteen.
struct SortChain {
    const hbf_access_t *acc; uint64_t n; const RangeSnap *ranges; const ModelParams *mp_dev; BatchCtrl *ctrl; DevState *state;
    uint64_t *keys0, *keys1, *terms; uint32_t *idx0, *idx1, *hist, *desc0, *desc1; void *scan_desc;
    uint8_t *status; int64_t *completion, *stall; const int64_t *busy; int64_t *busy_stage; hbf_die_stats_t *stats_stage;
    const unsigned long long *claim_limit; uint32_t *die_claims;
    uint32_t n_queues, n_dies; uint64_t desc_words, scan_words;
    unsigned cls_grid, hist_grid, sort_grid, scan_grid, stall_grid;
    const InTile *in_tile; uint32_t n_tiles;
};

__global__ void k_zero_words(uint32_t *p, uint64_t words) {
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < words; i += (uint64_t)gridDim.x * blockDim.x) p[i] = 0u;
}

// (MAY_SORT = false, for a context whose caller declares issue order: the same kernel without the device-side launches,
// which cost a kernel that contains them several microseconds even when none is made)
template <bool MAY_SORT>
__global__ void __launch_bounds__(256) k_after_inorder(const __grid_constant__ SortChain c) {
    if (c.ctrl->skip) return;                                // refused: nothing to do
    if (c.ctrl->inorder_used) {
        // served in issue order.  Stall total of the batch: per tile the exact sum if it was re-served, else the as-if
        // sum plus its corrections
        long long tot = 0;
        for (uint32_t t = threadIdx.x; t < c.n_tiles; t += blockDim.x) {
            const InTile v = c.in_tile[t];
            tot += v.reserve ? v.true_sum : v.spec_sum + v.fix_delta;
        }
        tot = warp_sum(tot);
        if ((threadIdx.x & 31) == 0 && tot) atomicAdd((unsigned long long *)&c.ctrl->modeled_ns, (unsigned long long)tot);
        return;
    }
    if constexpr (MAY_SORT) {
    if (!c.ctrl->run_sort || threadIdx.x != 0) return;
    cudaStream_t st = cudaStreamTailLaunch;
    k_begin<<<1, 1024, 0, st>>>(c.ctrl, c.state, c.busy, c.busy_stage, c.stats_stage, c.hist, c.n_queues, c.n_dies, 1, 1, c.die_claims);
    k_zero_words<<<(unsigned)min((unsigned long long)((c.desc_words + 1023) / 1024), 592ull), 1024, 0, st>>>(c.desc0, c.desc_words);
    k_zero_words<<<(unsigned)min((unsigned long long)((c.scan_words + 1023) / 1024), 592ull), 1024, 0, st>>>((uint32_t *)c.scan_desc, c.scan_words);
    k_classify<<<c.cls_grid, kClsThreads, 0, st>>>(c.acc, c.n, c.ranges, c.mp_dev, c.ctrl, c.keys0, c.terms, c.status, c.completion, c.stall);
    k_plan<<<1, 32, 0, st>>>(c.ctrl, 0);
    k_hist<<<c.hist_grid, kHistThreads, 0, st>>>(c.keys0, c.n, c.ctrl, c.hist);
    for (int p = 0; p < kMaxPasses; ++p)
        k_sort_pass<<<c.sort_grid, kSortThreads, kSortSmem, st>>>(p, c.n, c.ctrl, c.state, c.hist, c.keys0, c.keys1, c.idx0, c.idx1, c.desc0, c.desc1);
    k_scan<<<c.scan_grid, kScanThreads, 0, st>>>(c.terms, c.n, c.mp_dev, c.ctrl, c.state, c.keys0, c.keys1, c.idx0, c.idx1,
                                                 (ScanDesc *)c.scan_desc, c.busy, c.busy_stage, c.stats_stage, c.completion, c.stall,
                                                 c.claim_limit, c.die_claims);
    k_stalls<<<c.stall_grid, 256, 0, st>>>(c.acc, c.n, c.ctrl, c.completion, c.stall);
    }
}

static cudaError_t launch_after_inorder(const SubmitArgs &a, bool may_sort, cudaStream_t st) {
    const uint64_t n = a.n;
    const uint64_t sort_tiles = (n + kSortTile - 1) / kSortTile, scan_tiles = (n + kScanTile - 1) / kScanTile;
    cudaError_t e = ensure_dyn_smem((const void *)k_sort_pass, kSortSmem);   // (an attribute of the kernel: device-side launches use it too)
    if (e != cudaSuccess) return e;
    SortChain c{};
    c.acc = a.acc; c.n = n; c.ranges = a.ranges; c.mp_dev = a.mp_dev; c.ctrl = a.ctrl; c.state = a.state;
    c.keys0 = a.ws.keys[0]; c.keys1 = a.ws.keys[1]; c.terms = a.ws.terms; c.idx0 = a.ws.idx[0]; c.idx1 = a.ws.idx[1]; c.hist = a.ws.hist;
    c.desc0 = a.ws.sort_desc[0]; c.desc1 = a.ws.sort_desc[1]; c.scan_desc = a.ws.scan_desc;
    c.status = a.status; c.completion = a.completion; c.stall = a.stall; c.busy = a.busy; c.busy_stage = a.busy_stage;
    c.stats_stage = a.stats_stage; c.claim_limit = a.claim_limit; c.die_claims = a.die_claims;
    c.n_queues = a.mp.n_queues; c.n_dies = a.mp.n_dies;
    c.desc_words = sort_tiles * kRadix; c.scan_words = scan_tiles * (sizeof(ScanDesc) / 4);
    c.cls_grid = (unsigned)std::min<uint64_t>((n + kClsTile - 1) / kClsTile, (uint64_t)a.sm_count * 8);
    c.hist_grid = (unsigned)std::min<uint64_t>((n + kHistThreads * 8 - 1) / (kHistThreads * 8), (uint64_t)a.sm_count * 4);
    c.sort_grid = (unsigned)std::min<uint64_t>(sort_tiles, (uint64_t)a.sm_count * 3);
    c.scan_grid = (unsigned)std::min<uint64_t>(scan_tiles, (uint64_t)a.sm_count * 8);
    c.stall_grid = (unsigned)std::max<uint64_t>(1, std::min<uint64_t>((n + 255) / 256, (uint64_t)a.sm_count * 16));
    const InTileMap tmap = inorder_tile_map(n, a.sm_count, a.bal && a.bal->on && a.bal->dev);
    c.in_tile = reinterpret_cast<const InTile *>(a.ws.in_tile);
    c.n_tiles = inorder_small_batch(n) ? inorder_small_blocks(a.mp.n_queues) : tmap.n_tiles;
    if (may_sort) k_after_inorder<true><<<1, 256, 0, st>>>(c); else k_after_inorder<false><<<1, 256, 0, st>>>(c);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

// Kernel order of one batch.  AUTO: begin, the in-order kernels (they serve the batch when its records
// arrive in non-decreasing issue order), one thread that launches the sort kernels from the device if the
// in-order attempt handed the batch over, finish.  SORT / SORT_FULL: begin, sort kernels, finish.
cudaError_t launch_submit(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    auto mark = [&](int k) { if (a.ev) cudaEventRecord(a.ev[k], st); };
    const bool try_inorder = a.inorder_ok && (a.path == HBF_PATH_AUTO || a.path == HBF_PATH_INORDER);
    const bool sort_kernels = a.path != HBF_PATH_INORDER || !a.inorder_ok;
    {
        const void *small[] = {(const void *)k_begin, (const void *)k_finish};
        for (const void *f : small) { cudaError_t e = ensure_dyn_smem(f, 0); if (e != cudaSuccess) return e; }
    }
    mark(0);
    k_begin<<<1, 1024, 0, st>>>(a.ctrl, a.state, a.busy, a.busy_stage, a.stats_stage, a.ws.hist, a.mp.n_queues, a.mp.n_dies,
                               0, try_inorder ? 0 : 1, a.die_claims);
    g_kernel_launches += 1;
    if (n > 0) {
        if (try_inorder) {
            mark(7);
            cudaError_t e = launch_inorder(a, st);
            if (e != cudaSuccess) return e;
            mark(8);
            e = launch_after_inorder(a, sort_kernels, st);
            if (e != cudaSuccess) return e;
            mark(1); mark(2); mark(3); mark(4);
        } else {
            cudaError_t e = launch_sort_path(a, st);
            if (e != cudaSuccess) return e;
        }
    } else {
        mark(1); mark(2); mark(3); mark(4);
    }
    mark(5);
    const unsigned fin_grid = (unsigned)std::max<uint64_t>(1, std::min<uint64_t>((n + 1023) / 1024, (uint64_t)a.sm_count * 4));
    k_finish<<<fin_grid, 256, 0, st>>>(n, a.ctrl, a.state, a.busy, a.busy_stage, a.pending, a.stats_stage, a.die_stats,
                                       a.completion, a.stall, a.result, a.mp_dev, a.mp.n_queues, a.mp.n_dies, a.binned, a.bus_on);
    g_kernel_launches += 1;
    mark(6);
    return cudaGetLastError();
}

__global__ void k_add_stats(long long *total, const long long *part, uint32_t words) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < words) total[i] += part[i];
}
cudaError_t launch_add_stats(hbf_die_stats_t *total, const hbf_die_stats_t *part, uint32_t n_dies, cudaStream_t st) {
    const uint32_t words = n_dies * 6u;
    k_add_stats<<<(words + 255) / 256, 256, 0, st>>>(reinterpret_cast<long long *>(total), reinterpret_cast<const long long *>(part), words);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

__global__ void k_add_result(hbf_batch_result_t *sum, const hbf_batch_result_t *part, int first) {
    hbf_batch_result_t s = *sum; const hbf_batch_result_t r = *part;
    if (first) { s = r; }
    else {
        if (s.code == HBF_OK && r.code != HBF_OK) s.code = r.code;
        s.n_native += r.n_native; s.n_modeled += r.n_modeled; s.n_fault += r.n_fault;
        s.modeled_ns += r.modeled_ns; s.service_ns += r.service_ns;
        s.max_completion_ns = max(s.max_completion_ns, r.max_completion_ns);
    }
    *sum = s;
}
cudaError_t launch_add_result(hbf_batch_result_t *sum, const hbf_batch_result_t *part, int first, cudaStream_t st) {
    k_add_result<<<1, 1, 0, st>>>(sum, part, first);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_queue_order(const BatchCtrl *ctrl, const Workspace &ws, uint32_t *out, uint64_t n, cudaStream_t st) {
    if (n == 0) return cudaSuccess;
    k_queue_order<<<(unsigned)std::min<uint64_t>((n + 255) / 256, 1184), 256, 0, st>>>(ctrl, ws.idx[0], ws.idx[1], out, n);
    return cudaGetLastError();
}

}  // namespace hbf
