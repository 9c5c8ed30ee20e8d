// In-order path of hbf_submit_batch: serves a batch whose records arrive in non-decreasing issue order
// without a global sort.  In such a batch the (issue, index) order of every queue is plain index order,
// so the batch can be cut into a few hundred contiguous tiles and handled as reduce - scan - apply over
// vectors of per-queue max-plus maps:
//   reduce  every tile composes, per queue, the maps B -> max(B + s, a + s) of its accesses in index order
//           into one aggregate (S, M); it also classifies, writes status[], counts, and sums per-die bytes;
//   scan    one thread per queue walks the tiles in order: busy-until entering each tile, final busy-until;
//   apply   every tile re-reads its records and, starting from its entering busy-until vector, serves them
//           chunk by chunk; completions and stalls leave through shared memory in batch order.
// Every global access is coalesced (records in, results out); nothing waits on another thread block.
// Inside a chunk the per-queue order is recovered with a stable shared-memory radix sort of
// (queue, position) words and a segmented max-plus scan.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

constexpr int kInThreads = 256;
constexpr int kInItems = 8;
constexpr int kInChunk = kInThreads * kInItems;          // 2048 records
constexpr int kInWarps = kInThreads / 32;
constexpr int kInPosBits = 11;                           // position inside the chunk
constexpr int kInDigitBits = 6;
constexpr int kInBins = 1 << kInDigitBits;
constexpr int kInWorkBytes = kInChunk * 28;              // S 8 + M 8 + xfer/op 4 + two key buffers 2*4
static_assert(kInWorkBytes >= kInChunk * 24, "the raw records are staged in the work region");

struct InMap { int64_t S, M; int f; };
__device__ __forceinline__ InMap in_compose(const InMap &x, const InMap &y) {     // x earlier, y later
    if (y.f) return y;
    InMap r; r.f = x.f; r.S = x.S + y.S; r.M = max(x.M + y.S, y.M); return r;
}
__device__ __forceinline__ InMap in_shfl_up(const InMap &m, int o) {
    InMap r; r.S = __shfl_up_sync(0xffffffffu, m.S, o); r.M = __shfl_up_sync(0xffffffffu, m.M, o);
    r.f = __shfl_up_sync(0xffffffffu, m.f, o); return r;
}

// MODE 0 = reduce, MODE 1 = apply
template <int MODE>
__global__ void __launch_bounds__(kInThreads, 2)
k_inorder(const hbf_access_t *__restrict__ acc, uint64_t n, uint64_t tile_records, const RangeSnap *__restrict__ ranges_g,
          const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl, uint8_t *__restrict__ status, int64_t *__restrict__ in_agg,
          const int64_t *__restrict__ in_bin, hbf_die_stats_t *stats_stage, int64_t *__restrict__ completion,
          int64_t *__restrict__ stall) {
    extern __shared__ __align__(16) unsigned char in_smem[];
    __shared__ RangeSnap rs;
    __shared__ ModelParams mp;
    __shared__ uint32_t s_cnt[kInWarps * kInBins];
    __shared__ uint32_t s_bin_start[kInBins];
    __shared__ uint32_t s_bin_warp[2];
    __shared__ InMap s_warp_map[kInWarps];
    __shared__ long long s_red[2];

    if (ctrl->skip) return;
    if (MODE == 1 && (ctrl->run_sort || !ctrl->inorder_used)) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < (int)(sizeof(RangeSnap) / 4); i += kInThreads)
        reinterpret_cast<uint32_t *>(&rs)[i] = reinterpret_cast<const uint32_t *>(ranges_g)[i];
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kInThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    const uint32_t R = mp_g->n_queues, n_dies = mp_g->n_dies;

    // shared-memory carve-up
    uint64_t *raw = reinterpret_cast<uint64_t *>(in_smem);                        // [chunk*3], dead after the terms are in registers
    int64_t *sS = reinterpret_cast<int64_t *>(in_smem);                           // [chunk]  service; later the completion
    int64_t *sM = sS + kInChunk;                                                   // [chunk]  arrival + service; later the stall
    uint32_t *sX = reinterpret_cast<uint32_t *>(sM + kInChunk);                    // [chunk]  transfer ns | op << 31
    uint32_t *keyA = sX + kInChunk, *keyB = keyA + kInChunk;                       // [chunk] each
    unsigned char *fixed = in_smem + kInWorkBytes;
    int64_t *aggS = reinterpret_cast<int64_t *>(fixed);                            // reduce: [R] ; apply: busy-until [R]
    int64_t *aggM = aggS + R;                                                      // reduce only
    // reduce only, per die: charged bytes as low/high 32-bit halves (native 32-bit shared atomics), access counts
    uint32_t *st_br_lo = reinterpret_cast<uint32_t *>(aggM + R), *st_br_hi = st_br_lo + n_dies;
    uint32_t *st_bp_lo = st_br_hi + n_dies, *st_bp_hi = st_bp_lo + n_dies;
    uint32_t *st_nr = st_bp_hi + n_dies, *st_np = st_nr + n_dies;

    const uint32_t tile = blockIdx.x;
    const uint64_t tile_begin = (uint64_t)tile * tile_records;
    const uint64_t tile_end = min(n, tile_begin + tile_records);
    if (MODE == 0) {
        for (uint32_t r = tid; r < R; r += kInThreads) { aggS[r] = 0; aggM[r] = kNegInf; }
        for (uint32_t d = tid; d < n_dies * 6u; d += kInThreads) st_br_lo[d] = 0u;
    } else {
        for (uint32_t r = tid; r < R; r += kInThreads) aggS[r] = in_bin[(uint64_t)tile * R + r];
    }
    if (tid < 2) s_red[tid] = tid == 1 ? INT64_MIN : 0;

    // radix plan of the chunk sort: queue ids 0..R (R marks records that are not modeled)
    const uint32_t qbits = 32u - (uint32_t)__clz((int)R);
    const uint32_t n_pass = (qbits + kInDigitBits - 1) / kInDigitBits;
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const bool aligned16 = (reinterpret_cast<uintptr_t>(acc) & 15u) == 0;

    unsigned long long c_native = 0, c_ready = 0, c_fault = 0;
    unsigned c_unsorted = 0;
    long long sum_stall = 0, max_c = INT64_MIN;

    for (uint64_t cbase = tile_begin; cbase < tile_end; cbase += kInChunk) {
        const int cnt = (int)min((uint64_t)kInChunk, tile_end - cbase);
        __syncthreads();                                   // the work region is free again
        // ---- load: 16-byte coalesced loads of the 24-byte records ---------------------------------
        const uint64_t *src = reinterpret_cast<const uint64_t *>(acc + cbase);
        if (cnt == kInChunk && aligned16) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
            uint4 *d4 = reinterpret_cast<uint4 *>(raw);
#pragma unroll
            for (int k = 0; k < kInChunk * 24 / 16 / kInThreads; ++k) d4[tid + k * kInThreads] = __ldg(s4 + tid + k * kInThreads);
        } else {
            for (int i = tid; i < cnt * 3; i += kInThreads) raw[i] = __ldg(src + i);
        }
        __syncthreads();
        // ---- terms: classify, decode, service; warp-striped so that memory order = (item, lane) order ----
        uint32_t key[kInItems], xo[kInItems];
        int64_t S[kInItems], M[kInItems];
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = warp * (32 * kInItems) + j * 32 + lane;
            key[j] = (R << kInPosBits) | (uint32_t)e; xo[j] = 0u; S[j] = 0; M[j] = 0;
            if (e < cnt) {
                const uint64_t addr = raw[e * 3];
                const int64_t issue = (int64_t)raw[e * 3 + 1];
                const uint64_t bf = raw[e * 3 + 2];
                const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
                int g = 0;
                const int st = classify(rs, addr, issue, bytes, flags, &g);
                if (MODE == 0) {
                    int64_t prev;
                    if (e > 0) prev = (int64_t)raw[e * 3 - 2];
                    else prev = cbase > 0 ? acc[cbase - 1].issue_ns : INT64_MIN;
                    c_unsorted |= issue < prev ? 1u : 0u;
                    if (status) status[cbase + e] = (uint8_t)st;
                }
                if (st == HBF_ST_READY) {
                    const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
                    const Decoded d = decode(mp, off, bytes);
                    const uint32_t op = flags & 1u;
                    const Terms t = service_terms(mp, bytes, d.npages, op, q_ppm, div_q);
                    key[j] = (d.queue << kInPosBits) | (uint32_t)e;
                    S[j] = t.s; M[j] = issue + (op ? t.xfer : 0) + t.s;
                    xo[j] = (uint32_t)t.xfer | (op << 31);
                    if (MODE == 0) {
                        ++c_ready;
                        // charged bytes < 2^33: add the low word, carry into the high word when it wraps
                        const uint32_t lo = (uint32_t)t.cb, hi = (uint32_t)((uint64_t)t.cb >> 32);
                        uint32_t *plo = op ? st_bp_lo : st_br_lo, *phi = op ? st_bp_hi : st_br_hi;
                        atomicAdd(op ? &st_np[d.die] : &st_nr[d.die], 1u);
                        const uint32_t old = atomicAdd(&plo[d.die], lo);
                        const uint32_t carry = hi + ((old + lo) < old ? 1u : 0u);
                        if (carry) atomicAdd(&phi[d.die], carry);
                    }
                } else if (st == HBF_ST_NATIVE) {
                    S[j] = issue;                            // apply: completion = issue, stall = 0
                    if (MODE == 0) ++c_native;
                } else if (MODE == 0) {
                    ++c_fault;
                }
            }
        }
        __syncthreads();                                   // every raw record has been read
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = warp * (32 * kInItems) + j * 32 + lane;
            sS[e] = S[j]; sM[e] = M[j]; sX[e] = xo[j];
        }
        // ---- stable radix sort of (queue, position) words by queue -----------------------------------
        uint32_t shift = kInPosBits;
        for (uint32_t p = 0; p < n_pass; ++p) {
            const uint32_t width = qbits / n_pass + (p < qbits % n_pass ? 1u : 0u);
            const uint32_t dmask = (1u << width) - 1u;
            uint32_t *dst = (p & 1u) ? keyB : keyA;
            const uint32_t *srcb = (p & 1u) ? keyA : keyB;
            for (int i = tid; i < kInWarps * kInBins; i += kInThreads) s_cnt[i] = 0u;
            if (p > 0) {
#pragma unroll
                for (int j = 0; j < kInItems; ++j) key[j] = srcb[warp * (32 * kInItems) + j * 32 + lane];
            }
            __syncthreads();
            uint32_t rank[kInItems];
            uint32_t *wcnt = s_cnt + warp * kInBins;
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const uint32_t d = (key[j] >> shift) & dmask;
                const unsigned peers = __match_any_sync(0xffffffffu, d);
                const uint32_t before = wcnt[d];
                rank[j] = before + (uint32_t)__popc(peers & lanemask_lt());
                __syncwarp();
                if ((peers >> lane) <= 1u) wcnt[d] = before + (uint32_t)__popc(peers);
                __syncwarp();
            }
            __syncthreads();
            if (tid < kInBins) {                            // per bin: exclusive over warps, then exclusive over bins
                uint32_t run = 0;
#pragma unroll
                for (int w = 0; w < kInWarps; ++w) { const uint32_t c = s_cnt[w * kInBins + tid]; s_cnt[w * kInBins + tid] = run; run += c; }
                uint32_t incl = run;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
                if (lane == 31) s_bin_warp[warp] = incl;
                s_bin_start[tid] = incl - run;
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const uint32_t d = (key[j] >> shift) & dmask;
                const uint32_t pos = s_bin_start[d] + (d >= 32u ? s_bin_warp[0] : 0u) + wcnt[d] + rank[j];
                dst[pos] = key[j];
            }
            shift += width;
            __syncthreads();
        }
        const uint32_t *sorted = (n_pass & 1u) ? keyA : keyB;
        // ---- segmented max-plus scan over the sorted order (blocked: 8 consecutive positions per thread) ----
        uint32_t sk[kInItems];
        {
            const uint4 *k4 = reinterpret_cast<const uint4 *>(sorted + tid * kInItems);
            const uint4 a = k4[0], b = k4[1];
            sk[0] = a.x; sk[1] = a.y; sk[2] = a.z; sk[3] = a.w; sk[4] = b.x; sk[5] = b.y; sk[6] = b.z; sk[7] = b.w;
        }
        const uint32_t prev_q = tid > 0 ? (sorted[tid * kInItems - 1] >> kInPosBits) : 0xffffffffu;
        const uint32_t next_q = tid < kInThreads - 1 ? (sorted[(tid + 1) * kInItems] >> kInPosBits) : 0xffffffffu;
        InMap tm; tm.f = 0; tm.S = 0; tm.M = kNegInf;
        {
            uint32_t pq = prev_q;
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const uint32_t q = sk[j] >> kInPosBits, e = sk[j] & (kInChunk - 1);
                S[j] = 0; M[j] = kNegInf;
                if (q < R) {
                    S[j] = sS[e]; M[j] = sM[e];
                    InMap el; el.S = S[j]; el.f = q != pq;
                    if (MODE == 1 && el.f) M[j] = max(aggS[q] + S[j], M[j]);      // head: enter with the queue's busy-until
                    el.M = M[j];
                    tm = in_compose(tm, el);
                }
                pq = q;
            }
        }
        InMap incl = tm;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const InMap up = in_shfl_up(incl, o); if (lane >= o) incl = in_compose(up, incl); }
        if (lane == 31) s_warp_map[warp] = incl;
        __syncthreads();
        InMap cur; cur.f = 0; cur.S = 0; cur.M = kNegInf;
        for (int w = 0; w < warp; ++w) cur = in_compose(cur, s_warp_map[w]);
        {
            InMap ex = in_shfl_up(incl, 1);
            if (lane == 0) { ex.f = 0; ex.S = 0; ex.M = kNegInf; }
            cur = in_compose(cur, ex);
        }
        {
            uint32_t pq = prev_q;
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const uint32_t q = sk[j] >> kInPosBits, e = sk[j] & (kInChunk - 1);
                if (q < R) {
                    InMap el; el.S = S[j]; el.M = M[j]; el.f = q != pq;
                    cur = in_compose(cur, el);
                    const uint32_t nq = j + 1 < kInItems ? (sk[j + 1] >> kInPosBits) : next_q;
                    if (MODE == 1) {
                        const uint32_t x = sX[e];
                        const int64_t xfer = (int64_t)(x & 0x7fffffffu);
                        const bool op = (x >> 31) != 0u;
                        const int64_t c = cur.M + (op ? 0 : xfer);
                        const int64_t issue = sM[e] - S[j] - (op ? xfer : 0);
                        sS[e] = c; sM[e] = c - issue;
                        sum_stall += c - issue; max_c = max(max_c, (long long)c);
                        if (nq != q) aggS[q] = cur.M;                               // last access of the queue in this chunk
                    } else if (nq != q) {
                        aggM[q] = max(aggM[q] + cur.S, cur.M); aggS[q] += cur.S;    // queue aggregate o chunk segment
                    }
                }
                pq = q;
            }
        }
        // ---- results leave in batch order ---------------------------------------------------------------
        if (MODE == 1) {
            __syncthreads();
            for (int e = tid; e < cnt; e += kInThreads) { completion[cbase + e] = sS[e]; stall[cbase + e] = sM[e]; }
        }
    }

    __syncthreads();
    if (MODE == 0) {
        longlong2 *out = reinterpret_cast<longlong2 *>(in_agg) + (uint64_t)tile * R;
        for (uint32_t r = tid; r < R; r += kInThreads) out[r] = make_longlong2(aggS[r], aggM[r]);
        for (uint32_t d = tid; d < n_dies; d += kInThreads) {
            unsigned long long *g = reinterpret_cast<unsigned long long *>(stats_stage + d);
            const unsigned long long br = ((unsigned long long)st_br_hi[d] << 32) | st_br_lo[d];
            const unsigned long long bp = ((unsigned long long)st_bp_hi[d] << 32) | st_bp_lo[d];
            if (br) atomicAdd(&g[1], br);
            if (bp) atomicAdd(&g[2], bp);
            if (st_nr[d]) atomicAdd(&g[4], (unsigned long long)st_nr[d]);
            if (st_np[d]) atomicAdd(&g[5], (unsigned long long)st_np[d]);
        }
        c_native = (unsigned long long)warp_sum((long long)c_native);
        c_ready = (unsigned long long)warp_sum((long long)c_ready);
        c_fault = (unsigned long long)warp_sum((long long)c_fault);
        c_unsorted = __any_sync(0xffffffffu, c_unsorted);
        if (lane == 0) {
            if (c_native) atomicAdd(&ctrl->n_native, c_native);
            if (c_ready) atomicAdd(&ctrl->n_ready, c_ready);
            if (c_fault) atomicAdd(&ctrl->n_fault, c_fault);
            if (c_unsorted) atomicOr(&ctrl->unsorted, 1u);
        }
    } else {
        sum_stall = warp_sum(sum_stall); max_c = warp_max(max_c);
        if (lane == 0) { atomicAdd((unsigned long long *)&s_red[0], (unsigned long long)sum_stall); atomicMax(&s_red[1], max_c); }
        __syncthreads();
        if (tid == 0) {
            atomicAdd((unsigned long long *)&ctrl->modeled_ns, (unsigned long long)s_red[0]);
            atomicMax(&ctrl->max_completion_ns, s_red[1]);
        }
    }
}

// scan over tiles, one thread per queue; also decides what happens to the batch
constexpr int kInScanThreads = 32;
constexpr int kInScanDepth = 16;

__global__ void __launch_bounds__(kInScanThreads)
k_inorder_scan(BatchCtrl *ctrl, const ModelParams *__restrict__ mp, uint32_t n_tiles, const int64_t *__restrict__ in_agg,
               int64_t *__restrict__ in_bin, const int64_t *__restrict__ busy, int64_t *busy_stage,
               hbf_die_stats_t *stats_stage, int forced) {
    __shared__ long long s_tot;
    if (ctrl->skip) return;
    const bool fault = ctrl->n_fault != 0, unsorted = ctrl->unsorted != 0u;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (fault) { ctrl->code = HBF_E_ACCESS_FAULT; ctrl->skip = 1; }                 // fail closed: refuse the batch
        else if (unsorted && forced) { ctrl->code = HBF_E_INVAL; ctrl->skip = 1; }
        else if (unsorted) ctrl->run_sort = 1u;                                         // hand the batch to the sort path
        else ctrl->inorder_used = 1u;
    }
    if (fault || unsorted) return;
    if (threadIdx.x == 0) s_tot = 0;
    __syncthreads();
    const uint32_t R = mp->n_queues;
    const uint32_t r = blockIdx.x * kInScanThreads + threadIdx.x;
    long long tot = 0;
    if (r < R) {
        int64_t B = busy[r];
        const longlong2 *a = reinterpret_cast<const longlong2 *>(in_agg) + r;
        uint32_t t = 0;
        for (; t + kInScanDepth <= n_tiles; t += kInScanDepth) {
            longlong2 v[kInScanDepth];
#pragma unroll
            for (int k = 0; k < kInScanDepth; ++k) v[k] = a[(uint64_t)(t + k) * R];
#pragma unroll
            for (int k = 0; k < kInScanDepth; ++k) { in_bin[(uint64_t)(t + k) * R + r] = B; B = max((int64_t)(B + v[k].x), (int64_t)v[k].y); tot += v[k].x; }
        }
        for (; t < n_tiles; ++t) {
            const longlong2 v = a[(uint64_t)t * R];
            in_bin[(uint64_t)t * R + r] = B; B = max((int64_t)(B + v.x), (int64_t)v.y); tot += v.x;
        }
        busy_stage[r] = B;
        const uint32_t die = mp->queue_level == 0u ? r / mp->planes : r;
        if (tot) atomicAdd(reinterpret_cast<unsigned long long *>(&stats_stage[die].busy_ns), (unsigned long long)tot);
    }
    tot = warp_sum(tot);
    if ((threadIdx.x & 31) == 0 && tot) atomicAdd((unsigned long long *)&s_tot, (unsigned long long)tot);
    __syncthreads();
    if (threadIdx.x == 0 && s_tot) atomicAdd((unsigned long long *)&ctrl->service_ns, (unsigned long long)s_tot);
}

uint64_t inorder_tile_records(uint64_t n, int sm_count) {
    const uint64_t want_tiles = std::min<uint64_t>(kInMaxTiles, (uint64_t)std::max(1, sm_count) * 4);
    uint64_t t = (n + want_tiles - 1) / want_tiles;
    t = (t + kInChunk - 1) / kInChunk * kInChunk;
    return std::max<uint64_t>(t, kInChunk);
}

cudaError_t launch_inorder(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    const uint64_t tile_records = inorder_tile_records(n, a.sm_count);
    const unsigned n_tiles = (unsigned)((n + tile_records - 1) / tile_records);
    const uint32_t R = a.mp.n_queues, nd = a.mp.n_dies;
    const size_t smem_reduce = (size_t)kInWorkBytes + (size_t)R * 16 + (size_t)nd * 24;
    const size_t smem_apply = (size_t)kInWorkBytes + (size_t)R * 8;
    static size_t set_reduce = 0, set_apply = 0;
    if (smem_reduce > set_reduce) {
        cudaError_t e = cudaFuncSetAttribute(k_inorder<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_reduce);
        if (e != cudaSuccess) return e;
        set_reduce = smem_reduce;
    }
    if (smem_apply > set_apply) {
        cudaError_t e = cudaFuncSetAttribute(k_inorder<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_apply);
        if (e != cudaSuccess) return e;
        set_apply = smem_apply;
    }
    k_inorder<0><<<n_tiles, kInThreads, smem_reduce, st>>>(a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.status, a.ws.in_agg,
                                                           a.ws.in_bin, a.stats_stage, a.completion, a.stall);
    k_inorder_scan<<<(R + kInScanThreads - 1) / kInScanThreads, kInScanThreads, 0, st>>>(
        a.ctrl, a.mp_dev, n_tiles, a.ws.in_agg, a.ws.in_bin, a.busy, a.busy_stage, a.stats_stage, a.path == HBF_PATH_INORDER ? 1 : 0);
    k_inorder<1><<<n_tiles, kInThreads, smem_apply, st>>>(a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.status, a.ws.in_agg,
                                                          a.ws.in_bin, a.stats_stage, a.completion, a.stall);
    g_kernel_launches += 3;
    return cudaGetLastError();
}

}  // namespace hbf
