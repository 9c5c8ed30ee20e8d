// Page-granular submit: every page a modeled access touches becomes a request of its own (decoded by its own
// first byte, one page of array time, the transfer of its own bytes), and the access completes with its last
// part.  The paper's back end is a page-based flash simulator; the splitting rule itself is this library's.
//   count   parts per access (1 for an access that is not modeled), summed per row of 32 accesses and per tile of 64 rows;
//           a row's parts-before-it within its tile are kept
//   scan    exclusive scan of the tile sums by one block; the total goes back to the host, which sizes the rest
//   expand  a warp per row, no block-wide step: the warp reads its 32 records, knows where its parts begin (tile offset
//           + row offset), and writes them, in (access, part) order, as ordinary access records
//   serve   the ordinary submit path runs on the part records (they keep the batch's issue order)
//   join    completion of an access = the latest completion of its parts; the batch summary counts accesses
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

constexpr int kPgThreads = 256;
constexpr int kPgItems = 8;
constexpr int kPgTile = kPgThreads * kPgItems;
constexpr int kPgRows = kPgTile / 32;                    // rows of 32 consecutive accesses per tile

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

// the same with the one registered range in the kernel's arguments: nothing is read from memory to classify
__device__ __forceinline__ uint32_t parts_of_fast(const FastRange &fr, uint32_t page_shift, uint64_t addr, int64_t issue, uint64_t bf,
                                                  uint32_t *first_bytes) {
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    const uint64_t rel = addr - fr.base;
    const uint32_t need = (flags & 1u) ? (uint32_t)HBF_PERM_PROGRAM : (uint32_t)HBF_PERM_READ;
    const bool ready = bytes != 0u && (flags & ~1u) == 0u && issue >= 0 && issue < HBF_ISSUE_LIMIT && addr >= fr.base &&
                       rel < fr.length && (uint64_t)bytes <= fr.length - rel && (fr.perms & need) != 0u;
    *first_bytes = bytes;
    if (!ready) return 1u;
    const uint32_t page = 1u << page_shift, in_page = (uint32_t)(fr.media_offset + rel) & (page - 1u);
    *first_bytes = min(bytes, page - in_page);
    return (uint32_t)(((uint64_t)in_page + bytes + page - 1u) >> page_shift);
}

__global__ void __launch_bounds__(kPgThreads)
k_paged_count(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp,
              unsigned long long *__restrict__ tile_sum, uint32_t *__restrict__ row_off) {
    __shared__ uint32_t s_row[kPgRows];
    const uint64_t base = (uint64_t)blockIdx.x * kPgTile;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#pragma unroll
    for (int j = 0; j < kPgItems; ++j) {                     // row j * 8 + warp of the tile: accesses base + 32 row .. + 31
        const uint64_t i = base + (uint64_t)(j * kPgThreads + tid);
        uint64_t fb;
        uint32_t c = i < n ? parts_of(*ranges, *mp, reinterpret_cast<const uint64_t *>(acc + i), &fb) : 0u;
        c = (uint32_t)warp_sum((long long)c);
        if (lane == 0) s_row[j * (kPgThreads / 32) + warp] = c;
    }
    __syncthreads();
    if (warp == 0) {                                         // exclusive scan of the 64 row sums: two per lane
        const uint32_t a = s_row[2 * lane], b = s_row[2 * lane + 1];
        uint32_t incl = a + b;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        const uint32_t before = incl - (a + b);
        uint32_t *ro = row_off + (uint64_t)blockIdx.x * kPgRows;
        ro[2 * lane] = before; ro[2 * lane + 1] = before + a;
        if (lane == 31) tile_sum[blockIdx.x] = incl;
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

// A warp per row of 32 consecutive accesses, rows dealt round-robin to the grid's warps; no block-wide step.  The warp
// reads its 768 bytes of records, scans the part counts with shuffles, and every lane writes the parts of its access,
// walking through the access page by page: the 32 accesses' parts are consecutive in the output, so a warp's stores of
// one round fall into one short stretch.  An access of more than kPgWide parts (a very large access) is cut by the
// whole warp, a part per lane.  The kernel is bound by instruction issue, not by its bytes, which is why the common
// case (one registered range, an access inside one page) is kept short.
constexpr uint32_t kPgWide = 8;
constexpr int kPgUnroll = 2;                             // rows whose loads a warp has in flight together
constexpr int kPgWaves = 4;                              // blocks of the expand grid per resident block slot

template <bool FAST>
__global__ void __launch_bounds__(kPgThreads)
k_paged_expand(const hbf_access_t *__restrict__ acc, uint64_t n, const RangeSnap *__restrict__ ranges, const ModelParams *__restrict__ mp,
               const FastRange fast, const uint32_t page_shift, const unsigned long long *__restrict__ tile_off,
               const uint32_t *__restrict__ row_off, uint64_t capacity, hbf_access_t *__restrict__ parts, uint32_t *__restrict__ part_first) {
    const int lane = threadIdx.x & 31;
    const uint64_t warps = (uint64_t)gridDim.x * (kPgThreads / 32), rows = (n + 31) / 32;
    const uint32_t page = 1u << page_shift;
    uint64_t *out = reinterpret_cast<uint64_t *>(parts);
    for (uint64_t row0 = (uint64_t)blockIdx.x * (kPgThreads / 32) + (threadIdx.x >> 5); row0 < rows; row0 += warps * kPgUnroll) {
        // the loads of kPgUnroll rows go out together
        uint64_t r_addr[kPgUnroll], r_issue[kPgUnroll], r_bf[kPgUnroll], r_at[kPgUnroll];
#pragma unroll
        for (int u = 0; u < kPgUnroll; ++u) {
            const uint64_t row = row0 + (uint64_t)u * warps, i = row * 32 + (uint64_t)lane;
            r_addr[u] = r_issue[u] = r_bf[u] = r_at[u] = 0ull;
            if (row < rows) r_at[u] = tile_off[row / kPgRows] + row_off[row];
            if (i < n) {
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
                r_addr[u] = __ldg(rec); r_issue[u] = __ldg(rec + 1); r_bf[u] = __ldg(rec + 2);
            }
        }
#pragma unroll
        for (int u = 0; u < kPgUnroll; ++u) {
        const uint64_t row = row0 + (uint64_t)u * warps;
        if (row >= rows) break;
        const uint64_t i = row * 32 + (uint64_t)lane;
        const bool have = i < n;
        const uint64_t addr = r_addr[u], issue = r_issue[u], bf = r_bf[u];
        uint32_t cnt = 0u, head = 0u;
        const uint64_t row_at = r_at[u];
        if (have) {
            if (FAST) cnt = parts_of_fast(fast, page_shift, addr, (int64_t)issue, bf, &head);
            else { uint64_t h; cnt = parts_of(*ranges, *mp, reinterpret_cast<const uint64_t *>(acc + i), &h); head = (uint32_t)h; }
        }
        uint32_t incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        const uint64_t at = row_at + (incl - cnt);
        if (have) part_first[i] = (uint32_t)at;
        if (i == n - 1) part_first[n] = (uint32_t)(at + cnt);
        // the host checked the total against the capacity before this launch; the tests on it only keep a wrong call harmless
        if (cnt == 1u) {
            if (at < capacity) { uint64_t *o = out + at * 3ull; o[0] = addr; o[1] = issue; o[2] = bf; }
        } else if (cnt > 1u && cnt <= kPgWide) {
            uint64_t *o = out + at * 3ull;
            uint64_t a = addr;
            uint32_t left = (uint32_t)bf, len = head;
            const uint64_t hi = bf & 0xffffffff00000000ull;
            for (uint32_t p = 0; p < cnt; ++p) {
                if (at + p < capacity) { o[0] = a; o[1] = issue; o[2] = hi | len; }
                o += 3; a += len; left -= len; len = min(left, page);
            }
        }
        unsigned wide = __ballot_sync(0xffffffffu, cnt > kPgWide);
        while (wide) {
            const int src = __ffs(wide) - 1;
            wide &= wide - 1u;
            const uint64_t a0 = __shfl_sync(0xffffffffu, addr, src), is = __shfl_sync(0xffffffffu, issue, src);
            const uint64_t b = __shfl_sync(0xffffffffu, bf, src), base_at = __shfl_sync(0xffffffffu, at, src);
            const uint32_t hd = __shfl_sync(0xffffffffu, head, src), c = __shfl_sync(0xffffffffu, cnt, src);
            for (uint32_t p = (uint32_t)lane; p < c; p += 32u) {
                const uint64_t skip = p == 0u ? 0ull : (uint64_t)hd + (uint64_t)(p - 1u) * page;
                const uint64_t len = p == 0u ? (uint64_t)hd : min((uint64_t)(uint32_t)b - skip, (uint64_t)page);
                if (base_at + p < capacity) {
                    uint64_t *o = out + (base_at + p) * 3ull;
                    o[0] = a0 + skip; o[1] = is; o[2] = (b & 0xffffffff00000000ull) | len;
                }
            }
        }
        }
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
    void *ts = take(tiles * 8), *ro = take(tiles * kPgRows * 4), *tot = take(sizeof(PagedSums) + 8), *pf = take((nn + 1) * 4);
    void *pa = take(cap * sizeof(hbf_access_t)), *pc = take(cap * 8), *ps = take(cap * 8), *pst = take(cap);
    const size_t inner = workspace_layout(cap, n_queues, nullptr, nullptr, with_bus);
    void *in = take(inner);
    if (pw) {
        pw->tile_sum = (unsigned long long *)ts; pw->row_off = (uint32_t *)ro; pw->total = (unsigned long long *)tot;
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
    k_paged_count<<<(unsigned)tiles, kPgThreads, 0, st>>>(acc, n, ranges, mp_dev, pw.tile_sum, pw.row_off);
    k_paged_tile_scan<<<1, 1024, 0, st>>>(pw.tile_sum, tiles, pw.total);
    g_kernel_launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_paged_expand(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev,
                                const FastRange &fast, uint32_t page_shift, uint64_t capacity, const PagedWorkspace &pw, int sm_count,
                                cudaStream_t st) {
    const uint64_t blocks = ((n + 31) / 32 + kPgThreads / 32 - 1) / (kPgThreads / 32);
    const unsigned grid = (unsigned)std::min<uint64_t>(blocks, (uint64_t)std::max(1, sm_count) * 8 * kPgWaves);
    if (fast.on)
        k_paged_expand<true><<<grid, kPgThreads, 0, st>>>(acc, n, ranges, mp_dev, fast, page_shift, pw.tile_sum, pw.row_off, capacity, pw.parts, pw.part_first);
    else
        k_paged_expand<false><<<grid, kPgThreads, 0, st>>>(acc, n, ranges, mp_dev, fast, page_shift, pw.tile_sum, pw.row_off, capacity, pw.parts, pw.part_first);
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
