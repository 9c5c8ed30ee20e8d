// Page-granular submit: every page a modeled access touches becomes a request of its own (decoded by its own
// first byte, one page of array time, the transfer of its own bytes), and the access completes with its last
// part.  The paper's back end is a page-based flash simulator; the splitting rule itself is this library's.
//   count   parts per access (1 for an access that is not modeled), summed per tile of 2,048 accesses
//   scan    exclusive scan of the tile sums by one block; the total goes back to the host, which sizes the rest
//   expand  every tile writes its accesses' parts, in (access, part) order, as ordinary access records
//   serve   the ordinary submit path runs on the part records (they keep the batch's issue order)
//   join    completion of an access = the latest completion of its parts; the batch summary counts accesses
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

constexpr int kPgThreads = 256;
constexpr int kPgItems = 8;
constexpr int kPgTile = kPgThreads * kPgItems;

// parts of one access: its pages when it is modeled, one (the record itself) otherwise
__device__ __forceinline__ uint32_t parts_of(const RangeSnap &rs, const ModelParams &mp, const uint64_t *rec, uint64_t *first_bytes) {
    const uint64_t addr = __ldg(rec), bf = __ldg(rec + 2);
    const int64_t issue = (int64_t)__ldg(rec + 1);
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    int g = 0;
    *first_bytes = bytes;
    if (classify(rs, addr, issue, bytes, flags, &g) != HBF_ST_READY) return 1u;
    const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
    const uint64_t page = 1ull << mp.page_shift, in_page = off & (page - 1ull);
    *first_bytes = min((uint64_t)bytes, page - in_page);     // bytes of the access that fall into its first page
    return (uint32_t)((in_page + bytes + page - 1ull) >> mp.page_shift);
}

__global__ void __launch_bounds__(kPgThreads)
k_paged_count(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp,
              unsigned long long *__restrict__ tile_sum) {
    __shared__ unsigned long long s_warp[kPgThreads / 32];
    const uint64_t base = (uint64_t)blockIdx.x * kPgTile;
    unsigned long long mine = 0;
#pragma unroll
    for (int j = 0; j < kPgItems; ++j) {
        const uint64_t i = base + (uint64_t)(j * kPgThreads + threadIdx.x);
        uint64_t fb;
        if (i < n) mine += parts_of(*ranges, *mp, reinterpret_cast<const uint64_t *>(acc + i), &fb);
    }
    mine = (unsigned long long)warp_sum((long long)mine);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long t = 0;
        for (int w = 0; w < kPgThreads / 32; ++w) t += s_warp[w];
        tile_sum[blockIdx.x] = t;
    }
}

// one block: tile sums -> exclusive offsets, in place; total[0] = number of parts of the batch
__global__ void __launch_bounds__(1024)
k_paged_tile_scan(unsigned long long *tile_sum, uint64_t n_tiles, unsigned long long *total) {
    __shared__ unsigned long long s_warp[32];
    __shared__ unsigned long long s_carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (uint64_t b = 0; b < n_tiles; b += 1024) {
        const uint64_t i = b + (uint64_t)tid;
        const unsigned long long v = i < n_tiles ? tile_sum[i] : 0ull;
        unsigned long long incl = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        unsigned long long before = s_carry;
        for (int w = 0; w < warp; ++w) before += s_warp[w];
        if (i < n_tiles) tile_sum[i] = before + incl - v;
        __syncthreads();
        if (tid == 1023) s_carry = before + incl;
        __syncthreads();
    }
    if (tid == 0) *total = s_carry;
}

// A tile first lays out where the parts of each of its accesses go (thread t takes kPgItems consecutive accesses,
// block scan of the counts); then the threads walk the tile's OUTPUT slots, consecutive threads writing
// consecutive part records: each finds its access by binary search in the tile's offsets and cuts its part out.
__global__ void __launch_bounds__(kPgThreads)
k_paged_expand(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp,
               const unsigned long long *__restrict__ tile_off, uint64_t capacity, hbf_access_t *__restrict__ parts,
               uint32_t *__restrict__ part_first) {
    __shared__ unsigned long long s_warp[kPgThreads / 32];
    __shared__ uint32_t s_first[kPgTile + 1];               // first part of every access of the tile, relative to the tile's first
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint64_t tile_base = (uint64_t)blockIdx.x * kPgTile;
    const uint32_t in_tile = (uint32_t)min((uint64_t)kPgTile, n - tile_base);
    const uint64_t first = tile_base + (uint64_t)tid * kPgItems;
    uint32_t cnt[kPgItems];
    unsigned long long mine = 0;
#pragma unroll
    for (int j = 0; j < kPgItems; ++j) {
        uint64_t fb;
        cnt[j] = first + j < n ? parts_of(*ranges, *mp, reinterpret_cast<const uint64_t *>(acc + first + j), &fb) : 0u;
        mine += cnt[j];
    }
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    unsigned long long local = incl - mine;
    for (int w = 0; w < warp; ++w) local += s_warp[w];
    const unsigned long long off0 = tile_off[blockIdx.x];
#pragma unroll
    for (int j = 0; j < kPgItems; ++j) {
        if (first + j < n) {
            s_first[tid * kPgItems + j] = (uint32_t)local;
            part_first[first + j] = (uint32_t)(off0 + local);
            local += cnt[j];
        }
    }
    unsigned long long tile_total = 0;
    for (int w = 0; w < kPgThreads / 32; ++w) tile_total += s_warp[w];
    if (tid == 0) {
        s_first[in_tile] = (uint32_t)tile_total;
        if (tile_base + in_tile == n) part_first[n] = (uint32_t)(off0 + tile_total);     // the tile that holds the last access
    }
    __syncthreads();
    const uint64_t page = 1ull << mp->page_shift;
    for (unsigned long long k = (unsigned long long)tid; k < tile_total; k += kPgThreads) {
        uint32_t lo = 0, hi = in_tile;                       // last access e with s_first[e] <= k
        while (hi - lo > 1u) { const uint32_t mid = (lo + hi) >> 1; if ((unsigned long long)s_first[mid] <= k) lo = mid; else hi = mid; }
        const uint32_t e = lo, part = (uint32_t)(k - s_first[e]), of = s_first[e + 1] - s_first[e];
        hbf_access_t r = acc[tile_base + e];
        if (of > 1u) {                                       // a modeled access of several pages
            int g = 0;
            classify(*ranges, r.addr, r.issue_ns, r.bytes, r.flags, &g);
            const uint64_t off = ranges->media_offset[g] + (r.addr - ranges->base[g]);
            const uint64_t head = page - (off & (page - 1ull));          // bytes in its first page
            const uint64_t skip = part == 0u ? 0ull : head + (uint64_t)(part - 1u) * page;
            const uint64_t len = part == 0u ? head : min((uint64_t)r.bytes - skip, page);
            r.addr += skip; r.bytes = (uint32_t)len;
        }
        if (off0 + k < capacity) parts[off0 + k] = r;       // the host checked the total against the capacity before this launch
    }
}

struct PagedSums { unsigned long long n_ready, stall_sum; };

__global__ void __launch_bounds__(256)
k_paged_join(uint64_t n, const uint32_t *__restrict__ part_first, const int64_t *__restrict__ part_completion,
             const int64_t *__restrict__ part_stall, const uint8_t *__restrict__ part_status,
             const hbf_batch_result_t *__restrict__ result, int64_t *__restrict__ completion, int64_t *__restrict__ stall,
             uint8_t *__restrict__ status, PagedSums *sums) {
    const bool served = result->code == HBF_OK;
    unsigned long long ready = 0;
    long long stall_sum = 0;
    for (uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint32_t lo = part_first[i], hi = part_first[i + 1];
        const uint8_t st = part_status[lo];
        if (status && (served || result->code == HBF_E_ACCESS_FAULT)) status[i] = st;   // a batch refused before classification leaves it alone
        int64_t done = 0, waited = 0;
        if (served) {
            done = part_completion[lo];
            for (uint32_t k = lo + 1; k < hi; ++k) done = max(done, part_completion[k]);
            // every part carries the access's issue time: completion - stall of the first part gives it back
            if (st == HBF_ST_READY) { waited = done - (part_completion[lo] - part_stall[lo]); ++ready; stall_sum += waited; }
        }
        completion[i] = done; stall[i] = waited;
    }
    ready = (unsigned long long)warp_sum((long long)ready); stall_sum = warp_sum(stall_sum);
    if ((threadIdx.x & 31) == 0) {
        if (ready) atomicAdd(&sums->n_ready, ready);
        if (stall_sum) atomicAdd(&sums->stall_sum, (unsigned long long)stall_sum);
    }
}

// the summary counts accesses, not parts
__global__ void k_paged_finish(hbf_batch_result_t *result, const PagedSums *sums) {
    if (result->code == HBF_OK) { result->n_modeled = sums->n_ready; result->modeled_ns = (int64_t)sums->stall_sum; }
}

size_t paged_layout(uint64_t n, uint64_t capacity, uint32_t n_queues, PagedWorkspace *pw, void *base_ptr, int with_bus) {
    const uint64_t nn = n ? n : 1, cap = capacity ? capacity : 1;
    const uint64_t tiles = (nn + kPgTile - 1) / kPgTile;
    size_t off = 0;
    char *b = static_cast<char *>(base_ptr);
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return b ? b + o : nullptr; };
    void *ts = take(tiles * 8), *tot = take(sizeof(PagedSums) + 8), *pf = take((nn + 1) * 4);
    void *pa = take(cap * sizeof(hbf_access_t)), *pc = take(cap * 8), *ps = take(cap * 8), *pst = take(cap);
    const size_t inner = workspace_layout(cap, n_queues, nullptr, nullptr, with_bus);
    void *in = take(inner);
    if (pw) {
        pw->tile_sum = (unsigned long long *)ts; pw->total = (unsigned long long *)tot;
        pw->sums = (void *)((char *)tot + (tot ? 8 : 0)); pw->part_first = (uint32_t *)pf;
        pw->parts = (hbf_access_t *)pa; pw->part_completion = (int64_t *)pc; pw->part_stall = (int64_t *)ps; pw->part_status = (uint8_t *)pst;
        pw->inner = in; pw->inner_bytes = inner; pw->bytes = off;
    }
    return off;
}

cudaError_t launch_paged_count(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev,
                               const PagedWorkspace &pw, cudaStream_t st) {
    const uint64_t tiles = (n + kPgTile - 1) / kPgTile;
    cudaError_t e = cudaMemsetAsync(pw.total, 0, sizeof(PagedSums) + 8, st);
    if (e != cudaSuccess) return e;
    k_paged_count<<<(unsigned)tiles, kPgThreads, 0, st>>>(acc, n, ranges, mp_dev, pw.tile_sum);
    k_paged_tile_scan<<<1, 1024, 0, st>>>(pw.tile_sum, tiles, pw.total);
    g_kernel_launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_paged_expand(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev,
                                uint64_t capacity, const PagedWorkspace &pw, cudaStream_t st) {
    const uint64_t tiles = (n + kPgTile - 1) / kPgTile;
    k_paged_expand<<<(unsigned)tiles, kPgThreads, 0, st>>>(acc, n, ranges, mp_dev, pw.tile_sum, capacity, pw.parts, pw.part_first);
    g_kernel_launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_paged_join(const hbf_access_t *acc, uint64_t n, const PagedWorkspace &pw, hbf_batch_result_t *result,
                              int64_t *completion, int64_t *stall, uint8_t *status, int sm_count, cudaStream_t st) {
    const unsigned grid = (unsigned)std::min<uint64_t>((n + 255) / 256, (uint64_t)std::max(1, sm_count) * 8);
    k_paged_join<<<grid, 256, 0, st>>>(n, pw.part_first, pw.part_completion, pw.part_stall, pw.part_status, result, completion, stall, status,
                                      reinterpret_cast<PagedSums *>(pw.sums));
    k_paged_finish<<<1, 1, 0, st>>>(result, reinterpret_cast<const PagedSums *>(pw.sums));
    g_kernel_launches += 2;
    return cudaGetLastError();
}

}  // namespace hbf
