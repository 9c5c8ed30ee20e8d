// In-order path of hbf_submit_batch: serves a batch whose records arrive in non-decreasing issue order
// without a global sort.  In such a batch the (issue, index) order of every queue is plain index order,
// so the batch can be cut into a few hundred contiguous tiles and handled as reduce - scan - apply over
// vectors of per-queue max-plus maps:
//   reduce  every tile classifies and decodes its records, writes status[], counts, sums per-die bytes,
//           and composes, per queue, the maps B -> max(B + s, a + s) of its accesses in index order into
//           one aggregate (S, M).  It also leaves a 24-byte "served image" of every record in the
//           workspace: service, arrival + service, transfer time, queue and the record's place in its
//           chunk's queue-major order, so that the apply pass repeats none of this work;
//   scan    one thread per queue walks the tiles in order: busy-until entering each tile, final busy-until;
//   apply   every tile reads its images and, starting from its entering busy-until vector, serves them
//           chunk by chunk; completions and stalls leave through shared memory in batch order.
// Every global access is coalesced; nothing waits on another thread block.
//
// Inside a 2,048-record chunk the records are bucketed by queue in shared memory: one atomic per record
// takes a slot in its queue's bucket, an exclusive scan of the per-queue counts gives the bucket starts,
// and each record then finds its index-order rank inside its (short) bucket by counting the smaller
// positions.  A chunk with a long bucket is bucketed by a stable radix sort instead.  Thread t serves
// the consecutive queues [t*qpt, (t+1)*qpt) one access after the other.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

constexpr int kInThreads = 256;
constexpr int kInItems = 8;
constexpr int kInChunk = kInThreads * kInItems;          // 2048 records
constexpr int kInWarps = kInThreads / 32;
constexpr int kInDigitBits = 6;
constexpr int kInBins = 1 << kInDigitBits;
constexpr int kInMaxBucket = 16;                         // longer buckets take the radix route
constexpr uint32_t kInNoQueue = 0xffffu;                 // record is not modeled (native or refused)
constexpr int kInSlotBytes = kInChunk * 24;
constexpr int kInCntBytes = (kInMaxQueues + 64) * 4;
constexpr int kInPosBytes = kInChunk * 2;
constexpr int kInStartRow = kInThreads + 8;              // u16 per chunk: first sorted position of each thread's queues, + end

// word 2 of a served image: transfer ns (31 bits) | op << 31 | queue << 32 | place in the chunk's queue-major order << 48
__device__ __forceinline__ uint32_t img_queue(uint64_t w2) { return (uint32_t)(w2 >> 32) & 0xffffu; }
__device__ __forceinline__ uint32_t img_place(uint64_t w2) { return (uint32_t)(w2 >> 48); }

// state arrays are laid out so that thread t's queues sit in different banks than thread t+1's
__device__ __forceinline__ uint32_t state_index(uint32_t q, uint32_t qpt_shift) {
    return ((q & ((1u << qpt_shift) - 1u)) << 8) | (q >> qpt_shift);
}

// ======================================================================================================
// reduce
// ======================================================================================================
__global__ void __launch_bounds__(kInThreads, 2)
k_inorder_reduce(const hbf_access_t *__restrict__ acc, uint64_t n, uint64_t tile_records, const RangeSnap *__restrict__ ranges_g,
                 const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl, uint8_t *__restrict__ status, int64_t *__restrict__ in_agg,
                 uint64_t *__restrict__ in_img, uint16_t *__restrict__ in_start, hbf_die_stats_t *stats_stage) {
    extern __shared__ __align__(16) unsigned char in_smem[];
    __shared__ ModelParams mp;
    __shared__ uint32_t s_cnt[kInWarps * kInBins];        // radix route only
    __shared__ uint32_t s_bin_start[kInBins];
    __shared__ uint32_t s_bin_warp[2];
    __shared__ uint32_t s_warp_tot[kInWarps];
    __shared__ uint16_t s_tstart[kInStartRow];

    if (ctrl->skip) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const RangeSnap &rs = *ranges_g;                      // read through the cache: shared memory is needed elsewhere
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kInThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    const uint32_t R = mp_g->n_queues, n_dies = mp_g->n_dies;

    // slot e holds record e on arrival, then its served image (in place)
    uint64_t *slot = reinterpret_cast<uint64_t *>(in_smem);
    uint32_t *qcnt = reinterpret_cast<uint32_t *>(in_smem + kInSlotBytes);             // [R + 1] counts, then bucket starts
    uint16_t *posA = reinterpret_cast<uint16_t *>(in_smem + kInSlotBytes + kInCntBytes);
    uint16_t *posB = posA + kInChunk;                                                  // positions in queue-major order
    int64_t *aggS = reinterpret_cast<int64_t *>(posB + kInChunk);                      // [2048] per-queue aggregate of the tile
    int64_t *aggM = aggS + kInMaxQueues;
    uint32_t *st_br_lo = reinterpret_cast<uint32_t *>(aggM + kInMaxQueues), *st_br_hi = st_br_lo + n_dies;   // per die
    uint32_t *st_bp_lo = st_br_hi + n_dies, *st_bp_hi = st_bp_lo + n_dies;
    uint32_t *st_nr = st_bp_hi + n_dies, *st_np = st_nr + n_dies;

    const uint32_t tile = blockIdx.x;
    const uint64_t tile_begin = (uint64_t)tile * tile_records;
    const uint64_t tile_end = min(n, tile_begin + tile_records);

    // queues per thread, rounded up to a power of two
    uint32_t qpt_shift = 0;
    while (((uint32_t)kInThreads << qpt_shift) < R) ++qpt_shift;
    const uint32_t qpt = 1u << qpt_shift;

    for (uint32_t i = tid; i < kInMaxQueues; i += kInThreads) { aggS[i] = 0; aggM[i] = kNegInf; }
    for (uint32_t d = tid; d < n_dies * 6u; d += kInThreads) st_br_lo[d] = 0u;

    const uint32_t qbits = 32u - (uint32_t)__clz((int)R);
    const uint32_t n_pass = (qbits + kInDigitBits - 1) / kInDigitBits;
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const bool aligned16 = (reinterpret_cast<uintptr_t>(acc) & 15u) == 0;

    unsigned long long c_native = 0, c_ready = 0, c_fault = 0;
    unsigned c_unsorted = 0;

    for (uint64_t cbase = tile_begin; cbase < tile_end; cbase += kInChunk) {
        const int cnt = (int)min((uint64_t)kInChunk, tile_end - cbase);
        __syncthreads();                                   // the previous chunk has left shared memory
        // ---- load: 16-byte coalesced loads of the 24-byte records; clear the per-queue counts ----------
        const uint64_t *src = reinterpret_cast<const uint64_t *>(acc + cbase);
        if (cnt == kInChunk && aligned16) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
            uint4 *d4 = reinterpret_cast<uint4 *>(slot);
#pragma unroll
            for (int k = 0; k < kInChunk * 24 / 16 / kInThreads; ++k) d4[tid + k * kInThreads] = __ldg(s4 + tid + k * kInThreads);
        } else {
            for (int i = tid; i < cnt * 3; i += kInThreads) slot[i] = __ldg(src + i);
        }
        for (uint32_t q = tid; q <= R; q += kInThreads) qcnt[q] = 0u;
        __syncthreads();
        // ---- issue order, checked before the slots are reused ------------------------------------------
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = j * kInThreads + tid;
            if (e < cnt) {
                const int64_t issue = (int64_t)slot[e * 3 + 1];
                const int64_t prev = e > 0 ? (int64_t)slot[e * 3 - 2] : (cbase > 0 ? acc[cbase - 1].issue_ns : INT64_MIN);
                c_unsorted |= issue < prev ? 1u : 0u;
            }
        }
        __syncthreads();
        // ---- terms, in place: classify, decode, service; take a slot in the queue's bucket ----------------
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = j * kInThreads + tid;
            if (e < cnt) {
                const uint64_t addr = slot[e * 3];
                const int64_t issue = (int64_t)slot[e * 3 + 1];
                const uint64_t bf = slot[e * 3 + 2];
                const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
                int g = 0;
                const int st = classify(rs, addr, issue, bytes, flags, &g);
                if (status) status[cbase + e] = (uint8_t)st;
                uint64_t w0 = 0, w1 = 0, w2 = (uint64_t)kInNoQueue << 32;
                if (st == HBF_ST_READY) {
                    const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
                    const Decoded d = decode(mp, off, bytes);
                    const uint32_t op = flags & 1u;
                    const Terms t = service_terms(mp, bytes, d.npages, op, q_ppm, div_q);
                    const uint32_t o = atomicAdd(&qcnt[d.queue], 1u);
                    w0 = (uint64_t)t.s;
                    w1 = (uint64_t)(issue + (op ? t.xfer : 0) + t.s);
                    w2 = (uint64_t)((uint32_t)t.xfer | (op << 31)) | ((uint64_t)d.queue << 32) | ((uint64_t)o << 48);
                    ++c_ready;
                    // charged bytes < 2^33: add the low word, carry into the high word when it wraps
                    const uint32_t lo = (uint32_t)t.cb, hi = (uint32_t)((uint64_t)t.cb >> 32);
                    uint32_t *plo = op ? st_bp_lo : st_br_lo, *phi = op ? st_bp_hi : st_br_hi;
                    atomicAdd(op ? &st_np[d.die] : &st_nr[d.die], 1u);
                    const uint32_t old = atomicAdd(&plo[d.die], lo);
                    const uint32_t carry = hi + ((old + lo) < old ? 1u : 0u);
                    if (carry) atomicAdd(&phi[d.die], carry);
                } else if (st == HBF_ST_NATIVE) {
                    w0 = (uint64_t)issue;                    // apply: completion = issue, stall = 0
                    ++c_native;
                } else {
                    ++c_fault;
                }
                slot[e * 3] = w0; slot[e * 3 + 1] = w1; slot[e * 3 + 2] = w2;
            }
        }
        __syncthreads();
        // ---- bucket starts: exclusive scan of the counts in queue order; qcnt[R] = modeled records ---------
        int use_radix;
        {
            const uint32_t q0 = (uint32_t)tid * qpt;
            uint32_t c[8], tot = 0, longest = 0;
            if (qpt == 8u) {                               // full width: two 16-byte loads, free of bank conflicts
                const uint4 lo = *reinterpret_cast<const uint4 *>(qcnt + q0), hi = *reinterpret_cast<const uint4 *>(qcnt + q0 + 4);
                c[0] = lo.x; c[1] = lo.y; c[2] = lo.z; c[3] = lo.w; c[4] = hi.x; c[5] = hi.y; c[6] = hi.z; c[7] = hi.w;
            } else {
#pragma unroll
                for (int b = 0; b < 8; ++b) c[b] = ((uint32_t)b < qpt && q0 + b < R) ? qcnt[q0 + b] : 0u;
            }
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                if (q0 + b >= R) c[b] = 0u;
                longest = max(longest, c[b]);
                const uint32_t t = c[b]; c[b] = tot; tot += t;
            }
            uint32_t incl = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
            if (lane == 31) s_warp_tot[warp] = incl;
            use_radix = __syncthreads_or(longest > (uint32_t)kInMaxBucket);
            uint32_t woff = 0;
            for (int w = 0; w < warp; ++w) woff += s_warp_tot[w];
            const uint32_t base = woff + incl - tot;
            if (qpt == 8u) {
                *reinterpret_cast<uint4 *>(qcnt + q0) = make_uint4(base + c[0], base + c[1], base + c[2], base + c[3]);
                *reinterpret_cast<uint4 *>(qcnt + q0 + 4) = make_uint4(base + c[4], base + c[5], base + c[6], base + c[7]);
            } else {
#pragma unroll
                for (int b = 0; b < 8; ++b)
                    if ((uint32_t)b < qpt && q0 + b < R) qcnt[q0 + b] = base + c[b];
            }
            s_tstart[tid] = (uint16_t)base;
            if (tid == kInThreads - 1) { qcnt[R] = base + tot; s_tstart[kInThreads] = (uint16_t)(base + tot); }
        }
        __syncthreads();
        if (!use_radix) {
            // ---- short buckets: records go to the slot they took, then find their index-order rank ------------
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const int e = j * kInThreads + tid;
                if (e < cnt) {
                    const uint64_t w2 = slot[e * 3 + 2];
                    const uint32_t q = img_queue(w2);
                    if (q != kInNoQueue) posA[qcnt[q] + img_place(w2)] = (uint16_t)e;
                }
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < kInItems; ++j) {
                const int e = j * kInThreads + tid;
                if (e < cnt) {
                    const uint64_t w2 = slot[e * 3 + 2];
                    const uint32_t q = img_queue(w2);
                    if (q != kInNoQueue) {
                        const uint32_t st0 = qcnt[q], c = qcnt[q + 1] - st0;
                        uint32_t rank = 0;
                        for (uint32_t i = 0; i < c; ++i) rank += (uint32_t)posA[st0 + i] < (uint32_t)e ? 1u : 0u;
                        const uint32_t p = st0 + rank;
                        posB[p] = (uint16_t)e;
                        slot[e * 3 + 2] = (w2 & 0x0000ffffffffffffull) | ((uint64_t)p << 48);
                    }
                }
            }
        } else {
            // ---- a long bucket: stable radix sort of the positions by queue (6-bit digits, warp ranking) ----
            uint32_t shift = 0;
            for (uint32_t p = 0; p < n_pass; ++p) {
                const uint32_t width = qbits / n_pass + (p < qbits % n_pass ? 1u : 0u);
                const uint32_t dmask = (1u << width) - 1u;
                const bool to_b = ((n_pass - 1u - p) & 1u) == 0u;            // the last pass lands in posB
                uint16_t *dst = to_b ? posB : posA;
                const uint16_t *srcp = to_b ? posA : posB;
                for (int i = tid; i < kInWarps * kInBins; i += kInThreads) s_cnt[i] = 0u;
                uint32_t e_[kInItems], dig[kInItems], rank[kInItems];
                __syncthreads();
#pragma unroll
                for (int j = 0; j < kInItems; ++j) {
                    const int i = warp * (32 * kInItems) + j * 32 + lane;       // memory order = (item, lane) order
                    e_[j] = p == 0 ? (uint32_t)i : (uint32_t)srcp[i];
                    uint32_t q = R;                                                // not modeled: behind every queue
                    if ((int)e_[j] < cnt) { const uint32_t qq = img_queue(slot[e_[j] * 3 + 2]); if (qq != kInNoQueue) q = qq; }
                    dig[j] = (q >> shift) & dmask;
                }
                uint32_t *wcnt = s_cnt + warp * kInBins;
#pragma unroll
                for (int j = 0; j < kInItems; ++j) {
                    const unsigned peers = __match_any_sync(0xffffffffu, dig[j]);
                    const uint32_t before = wcnt[dig[j]];
                    rank[j] = before + (uint32_t)__popc(peers & lanemask_lt());
                    __syncwarp();
                    if ((peers >> lane) <= 1u) wcnt[dig[j]] = before + (uint32_t)__popc(peers);
                    __syncwarp();
                }
                __syncthreads();
                if (tid < kInBins) {
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
                    const uint32_t d = dig[j];
                    dst[s_bin_start[d] + (d >= 32u ? s_bin_warp[0] : 0u) + wcnt[d] + rank[j]] = (uint16_t)e_[j];
                }
                shift += width;
                __syncthreads();                           // the warp counters are cleared again by the next pass
            }
            const uint32_t modeled = qcnt[R];
            for (uint32_t k = tid; k < modeled; k += kInThreads) {
                const uint32_t e = posB[k];
                slot[e * 3 + 2] = (slot[e * 3 + 2] & 0x0000ffffffffffffull) | ((uint64_t)k << 48);
            }
        }
        __syncthreads();
        // ---- aggregate: thread t walks its queues' accesses, which are consecutive in queue-major order --------
        {
            const uint32_t k0 = s_tstart[tid], k1 = s_tstart[tid + 1];
            uint32_t cur = kInNoQueue, ci = 0;
            int64_t S = 0, M = kNegInf;
            for (uint32_t k = k0; k < k1; ++k) {
                const uint32_t e = posB[k];
                const int64_t s = (int64_t)slot[e * 3], m = (int64_t)slot[e * 3 + 1];
                const uint32_t q = img_queue(slot[e * 3 + 2]);
                if (q != cur) {
                    if (cur != kInNoQueue) { aggS[ci] = S; aggM[ci] = M; }
                    cur = q; ci = state_index(q, qpt_shift); S = aggS[ci]; M = aggM[ci];
                }
                M = max(M + s, m); S += s;                  // aggregate o access
            }
            if (cur != kInNoQueue) { aggS[ci] = S; aggM[ci] = M; }
        }
        __syncthreads();
        // ---- the served images and the threads' starts leave for the apply pass ----------------------------
        {
            uint64_t *dst = in_img + cbase * 3;
            if (cnt == kInChunk) {
                const uint4 *s4 = reinterpret_cast<const uint4 *>(slot);
                uint4 *d4 = reinterpret_cast<uint4 *>(dst);
#pragma unroll
                for (int k = 0; k < kInChunk * 24 / 16 / kInThreads; ++k) d4[tid + k * kInThreads] = s4[tid + k * kInThreads];
            } else {
                for (int i = tid; i < cnt * 3; i += kInThreads) dst[i] = slot[i];
            }
            uint16_t *row = in_start + (cbase / kInChunk) * kInStartRow;
            for (int i = tid; i <= kInThreads; i += kInThreads) row[i] = s_tstart[i];
        }
    }

    __syncthreads();
    {
        longlong2 *out = reinterpret_cast<longlong2 *>(in_agg) + (uint64_t)tile * R;
        for (uint32_t q = tid; q < R; q += kInThreads) { const uint32_t i = state_index(q, qpt_shift); out[q] = make_longlong2(aggS[i], aggM[i]); }
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
    }
}

// ======================================================================================================
// scan over tiles, one thread per queue; also decides what happens to the batch
// ======================================================================================================
constexpr int kInScanThreads = 32;
constexpr int kInScanDepth = 16;

__global__ void __launch_bounds__(kInScanThreads)
k_inorder_scan(BatchCtrl *ctrl, const ModelParams *__restrict__ mp, uint32_t n_tiles, const int64_t *__restrict__ in_agg,
               int64_t *__restrict__ in_bin, const int64_t *__restrict__ busy, int64_t *busy_stage,
               hbf_die_stats_t *stats_stage, int forced) {
    if (ctrl->skip) return;
    const bool fault = ctrl->n_fault != 0, unsorted = ctrl->unsorted != 0u;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (fault) { ctrl->code = HBF_E_ACCESS_FAULT; ctrl->skip = 1; }                 // fail closed: refuse the batch
        else if (unsorted && forced) { ctrl->code = HBF_E_INVAL; ctrl->skip = 1; }
        else if (unsorted) ctrl->run_sort = 1u;                                         // hand the batch to the sort path
        else ctrl->inorder_used = 1u;
    }
    if (fault || unsorted) return;
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
            for (int k = 0; k < kInScanDepth; ++k) {
                in_bin[(uint64_t)(t + k) * R + r] = B; B = max((int64_t)(B + v[k].x), (int64_t)v[k].y); tot += v[k].x;
            }
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
    if (threadIdx.x == 0 && tot) atomicAdd((unsigned long long *)&ctrl->service_ns, (unsigned long long)tot);
}

// ======================================================================================================
// apply
// ======================================================================================================
__global__ void __launch_bounds__(kInThreads, 3)
k_inorder_apply(uint64_t n, uint64_t tile_records, uint32_t R, BatchCtrl *ctrl, const uint64_t *__restrict__ in_img,
                const uint16_t *__restrict__ in_start, const int64_t *__restrict__ in_bin, int64_t *__restrict__ completion,
                int64_t *__restrict__ stall) {
    extern __shared__ __align__(16) unsigned char in_smem[];
    __shared__ uint16_t s_tstart[kInStartRow];
    __shared__ long long s_red[2];
    if (ctrl->skip || ctrl->run_sort || !ctrl->inorder_used) return;
    const int tid = threadIdx.x, lane = tid & 31;
    uint64_t *slot = reinterpret_cast<uint64_t *>(in_smem);
    uint16_t *pos = reinterpret_cast<uint16_t *>(in_smem + kInSlotBytes);
    int64_t *busy = reinterpret_cast<int64_t *>(in_smem + kInSlotBytes + kInPosBytes);        // [2048], state_index order

    const uint32_t tile = blockIdx.x;
    const uint64_t tile_begin = (uint64_t)tile * tile_records;
    const uint64_t tile_end = min(n, tile_begin + tile_records);
    uint32_t qpt_shift = 0;
    while (((uint32_t)kInThreads << qpt_shift) < R) ++qpt_shift;
    for (uint32_t q = tid; q < R; q += kInThreads) busy[state_index(q, qpt_shift)] = in_bin[(uint64_t)tile * R + q];
    if (tid < 2) s_red[tid] = tid == 1 ? INT64_MIN : 0;
    long long sum_stall = 0, max_c = INT64_MIN;

    for (uint64_t cbase = tile_begin; cbase < tile_end; cbase += kInChunk) {
        const int cnt = (int)min((uint64_t)kInChunk, tile_end - cbase);
        __syncthreads();
        const uint64_t *src = in_img + cbase * 3;
        if (cnt == kInChunk) {
            const uint4 *s4 = reinterpret_cast<const uint4 *>(src);
            uint4 *d4 = reinterpret_cast<uint4 *>(slot);
#pragma unroll
            for (int k = 0; k < kInChunk * 24 / 16 / kInThreads; ++k) d4[tid + k * kInThreads] = __ldg(s4 + tid + k * kInThreads);
        } else {
            for (int i = tid; i < cnt * 3; i += kInThreads) slot[i] = __ldg(src + i);
        }
        const uint16_t *row = in_start + (cbase / kInChunk) * kInStartRow;
        for (int i = tid; i <= kInThreads; i += kInThreads) s_tstart[i] = row[i];
        __syncthreads();
        // positions in queue-major order
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = j * kInThreads + tid;
            if (e < cnt) {
                const uint64_t w2 = slot[e * 3 + 2];
                if (img_queue(w2) != kInNoQueue) pos[img_place(w2)] = (uint16_t)e;
            }
        }
        __syncthreads();
        // serve: thread t walks the accesses of its queues one after the other
        {
            const uint32_t k0 = s_tstart[tid], k1 = s_tstart[tid + 1];
            uint32_t cur = kInNoQueue, ci = 0;
            int64_t B = 0;
            for (uint32_t k = k0; k < k1; ++k) {
                const uint32_t e = pos[k];
                const int64_t s = (int64_t)slot[e * 3], m = (int64_t)slot[e * 3 + 1];
                const uint64_t w2 = slot[e * 3 + 2];
                const uint32_t q = img_queue(w2);
                if (q != cur) {
                    if (cur != kInNoQueue) busy[ci] = B;
                    cur = q; ci = state_index(q, qpt_shift); B = busy[ci];
                }
                const int64_t xfer = (int64_t)((uint32_t)w2 & 0x7fffffffu);
                const bool op = (((uint32_t)w2) >> 31) != 0u;
                B = max(B + s, m);                          // busy-until after this access
                const int64_t done = B + (op ? 0 : xfer);
                const int64_t wait = done - (m - s - (op ? xfer : 0));
                slot[e * 3] = (uint64_t)done; slot[e * 3 + 1] = (uint64_t)wait;
                sum_stall += wait; max_c = max(max_c, (long long)done);
            }
            if (cur != kInNoQueue) busy[ci] = B;
        }
        __syncthreads();
        for (int e = tid; e < cnt; e += kInThreads) { completion[cbase + e] = (int64_t)slot[e * 3]; stall[cbase + e] = (int64_t)slot[e * 3 + 1]; }
    }
    sum_stall = warp_sum(sum_stall); max_c = warp_max(max_c);
    if (lane == 0) { atomicAdd((unsigned long long *)&s_red[0], (unsigned long long)sum_stall); atomicMax(&s_red[1], max_c); }
    __syncthreads();
    if (tid == 0) {
        atomicAdd((unsigned long long *)&ctrl->modeled_ns, (unsigned long long)s_red[0]);
        atomicMax(&ctrl->max_completion_ns, s_red[1]);
    }
}

uint64_t inorder_tile_records(uint64_t n, int sm_count) {
    const uint64_t want_tiles = std::min<uint64_t>(kInMaxTiles, (uint64_t)std::max(1, sm_count) * 4);
    uint64_t t = (n + want_tiles - 1) / want_tiles;
    t = (t + kInChunk - 1) / kInChunk * kInChunk;
    return std::max<uint64_t>(t, kInChunk);
}

size_t inorder_start_bytes(uint64_t n) { return ((n + kInChunk - 1) / kInChunk + 1) * kInStartRow * sizeof(uint16_t); }

cudaError_t launch_inorder(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    const uint64_t tile_records = inorder_tile_records(n, a.sm_count);
    const unsigned n_tiles = (unsigned)((n + tile_records - 1) / tile_records);
    const uint32_t R = a.mp.n_queues, nd = a.mp.n_dies;
    const size_t smem_reduce = (size_t)kInSlotBytes + kInCntBytes + 2 * kInPosBytes + (size_t)kInMaxQueues * 16 + (size_t)nd * 24;
    const size_t smem_apply = (size_t)kInSlotBytes + kInPosBytes + (size_t)kInMaxQueues * 8;
    static size_t set_reduce = 0, set_apply = 0;
    if (smem_reduce > set_reduce) {
        cudaError_t e = cudaFuncSetAttribute(k_inorder_reduce, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_reduce);
        if (e != cudaSuccess) return e;
        set_reduce = smem_reduce;
    }
    if (smem_apply > set_apply) {
        cudaError_t e = cudaFuncSetAttribute(k_inorder_apply, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_apply);
        if (e != cudaSuccess) return e;
        set_apply = smem_apply;
    }
    k_inorder_reduce<<<n_tiles, kInThreads, smem_reduce, st>>>(a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.status, a.ws.in_agg,
                                                               a.ws.in_img, a.ws.in_start, a.stats_stage);
    k_inorder_scan<<<(R + kInScanThreads - 1) / kInScanThreads, kInScanThreads, 0, st>>>(
        a.ctrl, a.mp_dev, n_tiles, a.ws.in_agg, a.ws.in_bin, a.busy, a.busy_stage, a.stats_stage, a.path == HBF_PATH_INORDER ? 1 : 0);
    k_inorder_apply<<<n_tiles, kInThreads, smem_apply, st>>>(n, tile_records, R, a.ctrl, a.ws.in_img, a.ws.in_start, a.ws.in_bin,
                                                             a.completion, a.stall);
    g_kernel_launches += 3;
    return cudaGetLastError();
}

}  // namespace hbf
