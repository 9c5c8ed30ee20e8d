// In-order path of hbf_submit_batch: serves a batch whose records arrive in non-decreasing issue order
// without a global sort.  In such a batch the (issue, index) order of every queue is plain index order,
// so the batch is cut into a few hundred contiguous tiles that are served independently, in one pass:
//   serve   every tile classifies and decodes its records, writes status[], counts, sums per-die bytes, and
//           serves its accesses AS IF every queue were idle when the tile begins; completions and stalls
//           leave through shared memory in batch order.  Per queue it also keeps the composition (S, M) of
//           the maps B -> max(B + s, a + s) of its accesses (M is exactly the busy-until of the as-if run),
//           and per chunk it leaves the queue-major order of the chunk in the workspace;
//   scan    one thread per queue walks the tiles' aggregates in order: the true busy-until entering each
//           tile, and the final busy-until;
//   fix-up  one thread per (tile, queue) starts from the true entering busy-until and re-serves that queue's
//           accesses of the tile in order, until it meets an access that arrives when the queue is idle:
//           from there on the as-if run and the true run coincide (busy-until is monotone in its start
//           value, so the as-if run was idle there too).  At moderate load this touches a few accesses
//           per (tile, queue); under overload it degrades to re-serving everything, still exactly.
// The serve pass is the only one that streams the batch: 24 B read and 16 B + 1 B written per access, plus
// 4 B of order information.  Every global access of it is coalesced; nothing waits on another thread block.
//
// Inside a chunk (4,096 records) the records are bucketed by queue in shared memory: one atomic per record
// takes a slot in its queue's bucket, an exclusive scan of the per-queue counts gives the bucket starts,
// and each record then finds its index-order rank inside its (short) bucket by counting the smaller
// positions.  A chunk with a long bucket is bucketed by a stable radix sort instead.  Thread t serves
// the queues whose first access of the chunk falls into its own positions of that order.
#include <algorithm>

#include "device_utils.cuh"

namespace hbf {

// Block shape of the serve kernel.  Measured on the 20 M capacity-mode batch (ms for the in-order group):
// 256 x 8 records, 2 blocks/SM: 0.88; 512 x 4, 2 blocks/SM: 0.92; 512 x 8, 1 block/SM: 0.77; 1024 x 4, 1 block/SM: 0.72.
// Larger chunks amortise the per-chunk work over the 2,048 queue bins; more warps hide shared-memory latency.
// With one block per SM nothing hides the chunk's load, so the records arrive by bulk asynchronous copy (TMA)
// into one of two buffers while the previous chunk is being served; two 3,072-record buffers fit, two 4,096 do not.
#ifndef HBF_IN_THREADS
#define HBF_IN_THREADS 768
#define HBF_IN_ITEMS 4
#define HBF_IN_BLOCKS 1
#endif
constexpr int kInThreads = HBF_IN_THREADS;               // threads of a serve block
constexpr int kInItems = HBF_IN_ITEMS;                   // records per thread and chunk
constexpr int kInBlocksPerSM = HBF_IN_BLOCKS;            // resident serve blocks per SM (shared memory decides)
constexpr int kInChunk = kInThreads * kInItems;          // 4096 records
constexpr int kInWarps = kInThreads / 32;
constexpr int kInDigitBits = 6;
constexpr int kInBins = 1 << kInDigitBits;
constexpr int kInGroup = 4;                              // accesses a thread loads at once while serving
constexpr int kInMaxBucket = 16;                         // longer buckets take the radix route
constexpr uint32_t kInNoQueue = 0xffffu;                 // record is not modeled (native or refused)
constexpr int kInSlotBytes = kInChunk * 24;
constexpr int kInCntBytes = (kInMaxQueues + 64) * 4;
constexpr int kInPosBytes = kInChunk * 2;

// word 2 of a slot: transfer ns (31 bits) | op << 31 | queue << 32 | slot taken in the queue's bucket << 48
__device__ __forceinline__ uint32_t img_queue(uint64_t w2) { return (uint32_t)(w2 >> 32) & 0xffffu; }
__device__ __forceinline__ uint32_t img_place(uint64_t w2) { return (uint32_t)(w2 >> 48); }

// One access, from its record: status, and for a modeled access its queue, die and service terms.
struct Served { int st; uint32_t queue, die, op; int64_t s, xfer, cb; };
__device__ __forceinline__ Served serve_terms(const RangeSnap &rs, const ModelParams &mp, uint64_t addr, int64_t issue,
                                              uint64_t bf, int64_t q_ppm, const Div64 &div_q) {
    Served r; r.queue = 0; r.die = 0; r.op = 0; r.s = 0; r.xfer = 0; r.cb = 0;
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    int g = 0;
    r.st = classify(rs, addr, issue, bytes, flags, &g);
    if (r.st == HBF_ST_READY) {
        const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
        const Decoded d = decode(mp, off, bytes);
        r.op = flags & 1u;
        const Terms t = service_terms(mp, bytes, d.npages, r.op, q_ppm, div_q);
        r.queue = d.queue; r.die = d.die; r.s = t.s; r.xfer = t.xfer; r.cb = t.cb;
    }
    return r;
}

// The same terms for the common configuration (one registered range, power-of-two geometry, no thermal
// scaling in force, transfer table present): 32-bit arithmetic wherever the values allow it.
struct FastRange { uint64_t base, length, media_offset; uint32_t perms, on; };
__device__ __forceinline__ Served serve_terms_fast(const FastRange &f, const ModelParams &mp, uint64_t addr, int64_t issue, uint64_t bf) {
    Served r; r.queue = 0; r.die = 0; r.op = 0; r.s = 0; r.xfer = 0; r.cb = 0;
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    const uint64_t rel = addr - f.base;                       // wraps to a huge value below the base
    if (bytes == 0u || (flags & ~1u) != 0u || (uint32_t)((uint64_t)issue >> 32) >= (1u << (kIssueBits - 32))) { r.st = HBF_ST_UNSUPPORTED; return r; }
    if (rel >= f.length) { r.st = HBF_ST_NATIVE; return r; }
    if ((uint64_t)bytes > f.length - rel) { r.st = HBF_ST_FAULT_PARTIAL; return r; }
    r.op = flags & 1u;
    if (!(f.perms & (1u << r.op))) { r.st = HBF_ST_FAULT_PERM; return r; }
    r.st = HBF_ST_READY;
    const uint64_t off = f.media_offset + rel;
    const uint32_t u = (uint32_t)(off >> mp.stripe_shift);    // only the low interleave bits are used
    const uint32_t ch = u & (mp.channels - 1u), di = (u >> mp.ch_shift) & (mp.dies - 1u);
    const uint32_t pl = (u >> (mp.ch_shift + mp.die_shift)) & (mp.planes - 1u);
    r.die = ch * mp.dies + di;
    r.queue = mp.queue_level == 0u ? r.die * mp.planes + pl : r.die;
    const uint32_t page_mask = (1u << mp.page_shift) - 1u;
    const uint32_t npages = (uint32_t)(((uint64_t)((uint32_t)off & page_mask) + bytes + page_mask) >> mp.page_shift);
    const uint32_t gs = r.op ? mp.prog_gran_shift : mp.read_gran_shift;
    const uint64_t cb = (((uint64_t)bytes + ((1ull << gs) - 1ull)) >> gs) << gs;
    r.cb = (int64_t)cb;
    r.xfer = cb <= (uint64_t)mp.xfer_tab_max_cb ? (int64_t)__ldg(mp.xfer_tab + (uint32_t)(cb >> mp.xfer_tab_shift))
                                                 : (int64_t)div64(cb * 1000ull + mp.chan_bytes_per_us - 1ull, mp.div_chan);
    r.s = (int64_t)npages * (r.op ? mp.t_prog_ns : mp.t_read_ns);
    return r;
}

// index of a queue's state in the shared-memory arrays
__device__ __forceinline__ uint32_t state_index(uint32_t q, uint32_t qpt_shift) {
    (void)qpt_shift;
    return q;
}

// per-tile bookkeeping of the stall total: as-if-idle sum, fix-up corrections, and the exact sum of a re-served tile
struct InTile { long long spec_sum, fix_delta, true_sum; uint32_t reserve; uint32_t stragglers; };
// The first kInHead accesses of every (tile, queue), as the serve pass saw them: all the fix-up needs in the common case.
constexpr int kInHead = 8;
struct InHead { int64_t m, s; uint32_t xo, idx; };       // arrival + service, service, transfer | op << 31, batch index

// ======================================================================================================
// serve.  RESERVE = false: the streaming pass over every tile, every queue taken as idle at the tile's start.
// RESERVE = true: only for tiles the fix-up flagged (a queue stayed backlogged far into the tile): the same
// pass from the true entering busy-until, writing the exact results and nothing else.
// ======================================================================================================
template <bool RESERVE>
__global__ void __launch_bounds__(kInThreads, kInBlocksPerSM)
k_inorder_serve(const hbf_access_t *__restrict__ acc, uint64_t n, uint64_t tile_records, const RangeSnap *__restrict__ ranges_g,
                const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl, uint8_t *__restrict__ status, int64_t *__restrict__ in_agg,
                uint16_t *__restrict__ in_pos, uint16_t *__restrict__ in_start, uint32_t row_stride,
                hbf_die_stats_t *stats_stage, int64_t *__restrict__ completion, int64_t *__restrict__ stall,
                const int64_t *__restrict__ in_bin, InTile *in_tile, InHead *__restrict__ in_head, uint8_t *__restrict__ in_headcnt) {
    extern __shared__ __align__(16) unsigned char in_smem[];
    __shared__ ModelParams mp;
    __shared__ uint32_t s_cnt[kInWarps * kInBins];        // radix route only
    __shared__ uint32_t s_bin_start[kInBins];
    __shared__ uint32_t s_bin_warp[2];
    __shared__ uint32_t s_warp_tot[kInWarps];
    __shared__ long long s_red[2];
    __shared__ FastRange s_fast;
    __shared__ uint32_t s_heads_full;                     // queues whose head entries are complete
    __shared__ __align__(8) uint64_t s_mbar[2];           // one per record buffer: completion of its bulk load

    if (ctrl->skip) return;
    if (RESERVE && (ctrl->run_sort || !ctrl->inorder_used || !in_tile[blockIdx.x].reserve)) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const RangeSnap &rs = *ranges_g;                      // read through the cache: shared memory is needed elsewhere
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kInThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    const uint32_t R = mp_g->n_queues, n_dies = mp_g->n_dies;
    if (tid == 0) {
        FastRange f; f.base = rs.base[0]; f.length = rs.length[0]; f.media_offset = rs.media_offset[0]; f.perms = rs.perms[0];
        f.on = (rs.count == 1u && mp_g->pow2_geom && mp_g->xfer_tab_max_cb != 0u && ctrl->q_ppm == 1000000) ? 1u : 0u;
        s_fast = f;
    }

    // slot e holds record e on arrival, then its served image (in place)
    uint64_t *slot_buf[2] = {reinterpret_cast<uint64_t *>(in_smem), reinterpret_cast<uint64_t *>(in_smem + kInSlotBytes)};
    uint32_t *qcnt = reinterpret_cast<uint32_t *>(in_smem + 2 * kInSlotBytes);         // [R + 1] counts, then bucket starts
    uint16_t *posA = reinterpret_cast<uint16_t *>(in_smem + 2 * kInSlotBytes + kInCntBytes);
    uint16_t *posB = posA + kInChunk;                                                  // positions in queue-major order
    int64_t *aggS = reinterpret_cast<int64_t *>(posB + kInChunk);                      // [queues] per-queue aggregate of the tile
    int64_t *aggM = aggS + kInMaxQueues;
    uint32_t *st_br_lo = reinterpret_cast<uint32_t *>(aggM + kInMaxQueues), *st_br_hi = st_br_lo + n_dies;   // per die
    uint32_t *st_bp_lo = st_br_hi + n_dies, *st_bp_hi = st_bp_lo + n_dies;
    uint32_t *st_nr = st_bp_hi + n_dies, *st_np = st_nr + n_dies;
    uint8_t *hfill = reinterpret_cast<uint8_t *>(st_np + n_dies);                  // head-table entries written per queue

    const uint32_t tile = blockIdx.x;
    const uint64_t tile_begin = (uint64_t)tile * tile_records;
    const uint64_t tile_end = min(n, tile_begin + tile_records);

    // queues per thread, rounded up to a power of two
    uint32_t qpt_shift = 0;
    while (((uint32_t)kInThreads << qpt_shift) < R) ++qpt_shift;
    const uint32_t qpt = 1u << qpt_shift;

    for (uint32_t i = tid; i < kInMaxQueues; i += kInThreads) { aggS[i] = 0; aggM[i] = kNegInf; }
    if (RESERVE) {
        __syncthreads();
        for (uint32_t q = tid; q < R; q += kInThreads) aggM[state_index(q, qpt_shift)] = in_bin[(uint64_t)blockIdx.x * R + q];
    } else {
        for (uint32_t d = tid; d < n_dies * 6u; d += kInThreads) st_br_lo[d] = 0u;
        for (uint32_t i = tid; i < kInMaxQueues; i += kInThreads) hfill[i] = 0;
    }

    const uint32_t qbits = 32u - (uint32_t)__clz((int)R);
    const uint32_t n_pass = (qbits + kInDigitBits - 1) / kInDigitBits;
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const bool aligned16 = (reinterpret_cast<uintptr_t>(acc) & 15u) == 0;

    unsigned long long c_native = 0, c_ready = 0, c_fault = 0;
    unsigned c_unsorted = 0;
    long long sum_stall = 0, max_c = INT64_MIN;

    if (tid < 2) s_red[tid] = tid == 1 ? INT64_MIN : 0;
    if (tid == 0) s_heads_full = 0u;

    // Full chunks of a 16-byte aligned batch arrive by bulk asynchronous copy; the last, partial chunk of a tile
    // and unaligned batches are loaded by the threads.
    constexpr uint32_t kChunkBytes = (uint32_t)kInChunk * 24u;
    auto prefetch = [&](uint64_t cb, uint32_t buf) {       // thread 0, after a block barrier that retired the buffer's last use
        if (aligned16 && cb < tile_end && tile_end - cb >= (uint64_t)kInChunk) {
            mbar_expect_tx(&s_mbar[buf], kChunkBytes);
            bulk_load(slot_buf[buf], acc + cb, kChunkBytes, &s_mbar[buf]);
        }
    };
    if (tid == 0) { mbar_init(&s_mbar[0], 1u); mbar_init(&s_mbar[1], 1u); }
    __syncthreads();
    if (tid == 0) prefetch(tile_begin, 0u);
    uint32_t parity_bits = 0u;                              // bit b: parity of buffer b's next completed phase
    uint32_t chunk_no = 0u;

    for (uint64_t cbase = tile_begin; cbase < tile_end; cbase += kInChunk, ++chunk_no) {
        const int cnt = (int)min((uint64_t)kInChunk, tile_end - cbase);
        const uint32_t buf = chunk_no & 1u;
        uint64_t *slot = slot_buf[buf];
        __syncthreads();                                   // the previous chunk has left shared memory
        if (tid == 0) prefetch(cbase + kInChunk, buf ^ 1u);   // the next chunk lands while this one is served
        // ---- load: bulk copy issued one chunk ahead, or 16-byte coalesced loads; clear the per-queue counts ----------
        const uint64_t *src = reinterpret_cast<const uint64_t *>(acc + cbase);
        if (cnt == kInChunk && aligned16) {
            const bool arrived = mbar_wait_bounded(&s_mbar[buf], (parity_bits >> buf) & 1u);
            parity_bits ^= 1u << buf;
            if (__syncthreads_or(arrived ? 0 : 1)) {       // the copy did not complete in time: give the batch up
                if (tid == 0) atomicExch(&ctrl->code, (int)HBF_E_TIMEOUT);
                mbar_wait_bounded(&s_mbar[buf ^ 1u], (parity_bits >> (buf ^ 1u)) & 1u);   // let the copy in flight land, within the same limit
                return;
            }
        } else {
            for (int i = tid; i < cnt * 3; i += kInThreads) slot[i] = __ldg(src + i);
        }
        for (uint32_t q = tid; q <= R; q += kInThreads) qcnt[q] = 0u;
        __syncthreads();
        // ---- terms, in place: classify, decode, service; take a slot in the queue's bucket.  Word 1 (the issue
        // time) stays as it is until the queues are served, so the issue-order check can read the neighbour's.
#pragma unroll
        for (int j = 0; j < kInItems; ++j) {
            const int e = j * kInThreads + tid;
            if (e < cnt) {
                const uint64_t addr = slot[e * 3];
                const int64_t issue = (int64_t)slot[e * 3 + 1];
                if (!RESERVE) {
                    const int64_t prev = e > 0 ? (int64_t)slot[e * 3 - 2] : (cbase > 0 ? acc[cbase - 1].issue_ns : INT64_MIN);
                    c_unsorted |= issue < prev ? 1u : 0u;
                }
                const Served v = s_fast.on ? serve_terms_fast(s_fast, mp, addr, issue, slot[e * 3 + 2])
                                           : serve_terms(rs, mp, addr, issue, slot[e * 3 + 2], q_ppm, div_q);
                if (!RESERVE && status) status[cbase + e] = (uint8_t)v.st;
                uint64_t w0 = 0, w2 = (uint64_t)kInNoQueue << 32;
                if (v.st == HBF_ST_READY) {
                    const uint32_t o = atomicAdd(&qcnt[v.queue], 1u);
                    w0 = (uint64_t)v.s;
                    w2 = (uint64_t)((uint32_t)v.xfer | (v.op << 31)) | ((uint64_t)v.queue << 32) | ((uint64_t)o << 48);
                    if (!RESERVE) {
                        ++c_ready;
                        // charged bytes < 2^33: add the low word, carry into the high word when it wraps
                        const uint32_t lo = (uint32_t)v.cb, hi = (uint32_t)((uint64_t)v.cb >> 32);
                        uint32_t *plo = v.op ? st_bp_lo : st_br_lo, *phi = v.op ? st_bp_hi : st_br_hi;
                        atomicAdd(v.op ? &st_np[v.die] : &st_nr[v.die], 1u);
                        const uint32_t old = atomicAdd(&plo[v.die], lo);
                        const uint32_t carry = hi + ((old + lo) < old ? 1u : 0u);
                        if (carry) atomicAdd(&phi[v.die], carry);
                    }
                } else if (v.st == HBF_ST_NATIVE) {
                    w0 = (uint64_t)issue;                    // native: completion = issue, stall = 0
                    ++c_native;
                } else {
                    ++c_fault;
                }
                slot[e * 3] = w0; slot[e * 3 + 2] = w2;
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
            if (tid == kInThreads - 1) qcnt[R] = base + tot;
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
                    else slot[e * 3 + 1] = 0;              // native or refused: no stall
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
                        if (c > 1u)
                            for (uint32_t i = 0; i < c; ++i) rank += (uint32_t)posA[st0 + i] < (uint32_t)e ? 1u : 0u;
                        posB[st0 + rank] = (uint16_t)e;
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
                    if ((int)e_[j] < cnt) {
                        const uint32_t qq = img_queue(slot[e_[j] * 3 + 2]);
                        if (qq != kInNoQueue) q = qq; else if (p == 0) slot[e_[j] * 3 + 1] = 0;     // native or refused: no stall
                    }
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
        }
        __syncthreads();
        // ---- serve.  In queue-major order a queue's accesses are consecutive.  Thread t takes positions
        // [8t, 8t+8) and serves every queue whose first access of the chunk lies there, to that queue's last
        // access (which may lie past 8t+8; the thread owning those positions skips them).  Every thread thus
        // does about eight accesses, and a queue is touched by one thread only.  Loads go four at a time: they
        // are independent, only the max-plus chain is serial.  M is the aggregate's constant term and, at the
        // same time, the busy-until of the as-if-idle run.
        {
            const uint32_t modeled = qcnt[R];
            const uint32_t p0 = (uint32_t)tid * kInItems;
            const bool heads_on = !RESERVE && s_heads_full < R;
            if (p0 < modeled) {
                uint32_t cur = kInNoQueue, hf = 0;
                bool mine = false;                            // the queue being served was opened by this thread
                int64_t S = 0, M = kNegInf;
                uint32_t prev_q = p0 > 0 ? img_queue(slot[(uint32_t)posB[p0 - 1] * 3 + 2]) : kInNoQueue;
                auto close_queue = [&]() {
                    aggS[cur] = S; aggM[cur] = M;
                    if (heads_on) {
                        if (hfill[cur] < (uint8_t)kInHead && hf == (uint32_t)kInHead) atomicAdd(&s_heads_full, 1u);
                        hfill[cur] = (uint8_t)hf;
                    }
                };
                auto serve_one = [&](uint32_t e, int64_t sv, int64_t issue, uint64_t w2) {
                    const uint32_t x = (uint32_t)w2;
                    const int64_t xfer = (int64_t)(x & 0x7fffffffu);
                    const bool op = (x >> 31) != 0u;
                    const int64_t m = issue + (op ? xfer : 0) + sv;          // arrival + service
                    if (heads_on && hf < (uint32_t)kInHead) {                 // among the first accesses of this queue in the tile
                        InHead h; h.m = m; h.s = sv; h.xo = x; h.idx = (uint32_t)(cbase + e);
                        in_head[((uint64_t)tile * kInHead + hf) * R + cur] = h;
                        ++hf;
                    }
                    M = max(M + sv, m); S += sv;                              // aggregate o access; M = busy-until after it
                    const int64_t done = M + (op ? 0 : xfer);
                    slot[e * 3] = (uint64_t)done; slot[e * 3 + 1] = (uint64_t)(done - issue);
                    sum_stall += done - issue; max_c = max(max_c, (long long)done);
                };
#pragma unroll
                for (int g = 0; g < kInItems / kInGroup; ++g) {
                    const uint32_t pg = p0 + g * kInGroup;
                    uint32_t e[kInGroup];
                    int64_t s_[kInGroup], i_[kInGroup];
                    uint64_t w2[kInGroup];
#pragma unroll
                    for (int j = 0; j < kInGroup; ++j) e[j] = pg + j < modeled ? (uint32_t)posB[pg + j] : 0u;
#pragma unroll
                    for (int j = 0; j < kInGroup; ++j) { s_[j] = (int64_t)slot[e[j] * 3]; i_[j] = (int64_t)slot[e[j] * 3 + 1]; w2[j] = slot[e[j] * 3 + 2]; }
#pragma unroll
                    for (int j = 0; j < kInGroup; ++j) {
                        if (pg + j < modeled) {
                            const uint32_t q = img_queue(w2[j]);
                            if (q != prev_q) {                                // first access of queue q in this chunk
                                if (mine) close_queue();
                                cur = q; mine = true; S = aggS[q]; M = aggM[q];
                                if (heads_on) hf = hfill[q];
                            }
                            if (mine) serve_one(e[j], s_[j], i_[j], w2[j]);
                            prev_q = q;
                        }
                    }
                }
                if (mine) {                                    // the last queue opened here may go on past this thread's positions
                    for (uint32_t p = p0 + kInItems; p < modeled; ++p) {
                        const uint32_t e = posB[p];
                        const uint64_t w2 = slot[e * 3 + 2];
                        if (img_queue(w2) != cur) break;
                        serve_one(e, (int64_t)slot[e * 3], (int64_t)slot[e * 3 + 1], w2);
                    }
                    close_queue();
                }
            }
        }
        __syncthreads();
        // ---- results leave in batch order; the chunk's queue-major order stays behind for the fix-up ----------
        for (int e = tid; e < cnt; e += kInThreads) { completion[cbase + e] = (int64_t)slot[e * 3]; stall[cbase + e] = (int64_t)slot[e * 3 + 1]; }
        if (!RESERVE) {
            const uint32_t modeled = qcnt[R];
            for (uint32_t k = tid; k < modeled; k += kInThreads) in_pos[cbase + k] = posB[k];
            uint16_t *row = in_start + (cbase / kInChunk) * row_stride;
            for (uint32_t q = tid; q <= R; q += kInThreads) row[q] = (uint16_t)qcnt[q];
        }
    }

    __syncthreads();
    if (!RESERVE) {
        longlong2 *out = reinterpret_cast<longlong2 *>(in_agg) + (uint64_t)tile * R;
        for (uint32_t q = tid; q < R; q += kInThreads) {
            const uint32_t i = state_index(q, qpt_shift);
            out[q] = make_longlong2(aggS[i], aggM[i]);
            in_headcnt[(uint64_t)tile * R + q] = hfill[q];
        }
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
    sum_stall = warp_sum(sum_stall); max_c = warp_max(max_c);
    if (lane == 0) { atomicAdd((unsigned long long *)&s_red[0], (unsigned long long)sum_stall); atomicMax(&s_red[1], max_c); }
    __syncthreads();
    if (tid == 0) {
        if (RESERVE) in_tile[tile].true_sum = s_red[0];
        else { InTile t; t.spec_sum = s_red[0]; t.fix_delta = 0; t.true_sum = 0; t.reserve = 0u; t.stragglers = 0u; in_tile[tile] = t; }
        atomicMax(&ctrl->max_completion_ns, s_red[1]);
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
// fix-up: the true run differs from the as-if-idle run only at the head of each (tile, queue)
// ======================================================================================================
constexpr int kInFixThreads = 128;

// Phase 1, one thread per (tile, queue): walk the head table.  A queue that is still backlogged after
// kInHead accesses is a straggler: it goes on a list for phase 2, or, when a tile has many of them (the
// batch arrived on queues that were far behind), the whole tile is flagged to be served again.
__global__ void __launch_bounds__(kInFixThreads)
k_inorder_fixup(uint32_t R, uint32_t n_tiles, BatchCtrl *ctrl, const int64_t *__restrict__ in_bin,
                const InHead *__restrict__ in_head, const uint8_t *__restrict__ in_headcnt, int64_t *completion, int64_t *stall,
                InTile *in_tile, uint32_t *in_list) {
    if (ctrl->skip || ctrl->run_sort || !ctrl->inorder_used) return;
    const uint64_t idx = (uint64_t)blockIdx.x * kInFixThreads + threadIdx.x;          // tile * R + queue
    long long max_c = INT64_MIN;
    if (idx < (uint64_t)n_tiles * R) {
        const uint32_t tile = (uint32_t)(idx / R);
        const uint32_t q = (uint32_t)(idx % R);
        const uint32_t c = in_headcnt[idx];
        int64_t B = in_bin[idx];                             // true busy-until of the queue entering the tile
        int64_t Bs = kNegInf;                                // busy-until of the as-if-idle run, to know what it wrote
        long long dstall = 0;
        bool settled = false;
        for (uint32_t k = 0; k < c; ++k) {
            const InHead h = in_head[((uint64_t)tile * kInHead + k) * R + q];
            if (B <= h.m - h.s) { settled = true; break; }   // idle on arrival: from here on the as-if run was right
            B += h.s;                                          // it waited for the queue: starts at B
            Bs = max(Bs + h.s, h.m);
            const bool op = (h.xo >> 31) != 0u;
            const int64_t xfer = (int64_t)(h.xo & 0x7fffffffu);
            const int64_t done = B + (op ? 0 : xfer);
            dstall += B - Bs;                                  // completion moved from Bs + post to B + post
            completion[h.idx] = done; stall[h.idx] = done - (h.m - h.s - (op ? xfer : 0));
            max_c = max(max_c, (long long)done);
        }
        if (dstall) atomicAdd((unsigned long long *)&in_tile[tile].fix_delta, (unsigned long long)dstall);
        if (!settled && c == (uint32_t)kInHead) {
            const uint32_t rank = atomicAdd(&in_tile[tile].stragglers, 1u);
            if (rank >= max(8u, R / 16u)) in_tile[tile].reserve = 1u;
            else in_list[1 + atomicAdd(&in_list[0], 1u)] = (uint32_t)idx;
        }
    }
    max_c = warp_max(max_c);
    if ((threadIdx.x & 31) == 0 && max_c != INT64_MIN) atomicMax(&ctrl->max_completion_ns, max_c);
}

// Phase 2, one warp per straggler: re-serve the queue's accesses of the tile from the records until an
// access arrives on an idle queue.  The lanes take 32 consecutive chunks at a time: each composes the
// maps of the queue's accesses in its chunk, a warp scan over the lanes gives the true busy-until
// entering every chunk, and each lane then re-serves its chunk.  Past the point where the queue falls
// idle the re-served values equal what is already there, so lanes need not agree on where to stop.
constexpr uint32_t kInLongBudget = 4096;                  // accesses re-served for one (tile, queue) before the tile is re-served whole

__global__ void __launch_bounds__(kInFixThreads)
k_inorder_fixup_long(const hbf_access_t *__restrict__ acc, uint64_t n, uint64_t tile_records,
                     const RangeSnap *__restrict__ ranges_g, const ModelParams *__restrict__ mp_g, BatchCtrl *ctrl,
                     const int64_t *__restrict__ in_bin, const uint16_t *__restrict__ in_pos, const uint16_t *__restrict__ in_start,
                     uint32_t row_stride, int64_t *completion, int64_t *stall, InTile *in_tile, const uint32_t *__restrict__ in_list) {
    __shared__ ModelParams mp;
    if (ctrl->skip || ctrl->run_sort || !ctrl->inorder_used) return;
    const RangeSnap &rs = *ranges_g;
    for (int i = threadIdx.x; i < (int)(sizeof(ModelParams) / 4); i += kInFixThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    __syncthreads();
    const uint32_t R = mp.n_queues, count = in_list[0];
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warp_global = (blockIdx.x * kInFixThreads + threadIdx.x) >> 5, n_warps = (gridDim.x * kInFixThreads) >> 5;
    long long max_c = INT64_MIN;
    for (uint32_t w = warp_global; w < count; w += n_warps) {
        const uint32_t idx = in_list[1 + w];
        const uint32_t tile = idx / R, q = idx % R;
        if (in_tile[tile].reserve) continue;
        int64_t B = in_bin[idx];                             // true busy-until entering the next group of chunks
        long long dstall = 0;
        const uint64_t tile_begin = (uint64_t)tile * tile_records, tile_end = min(n, tile_begin + tile_records);
        uint32_t served = 0;
        for (uint64_t gbase = tile_begin; gbase < tile_end; gbase += 32ull * kInChunk) {
            const uint64_t cbase = gbase + (uint64_t)lane * kInChunk;
            uint32_t k0 = 0, k1 = 0;
            if (cbase < tile_end) {
                const uint16_t *row = in_start + (cbase / kInChunk) * row_stride;
                k0 = row[q]; k1 = row[q + 1];
            }
            // this lane's chunk as one map B -> max(B + S, M)
            int64_t S = 0, M = kNegInf;
            for (uint32_t k = k0; k < k1; ++k) {
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + cbase + in_pos[cbase + k]);
                const int64_t issue = (int64_t)rec[1];
                const Served v = serve_terms(rs, mp, rec[0], issue, rec[2], q_ppm, div_q);
                M = max(M + v.s, issue + (v.op ? v.xfer : 0) + v.s); S += v.s;
            }
            // exclusive scan of the maps over the lanes, applied to B
            int64_t iS = S, iM = M;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int64_t uS = __shfl_up_sync(0xffffffffu, iS, o), uM = __shfl_up_sync(0xffffffffu, iM, o);
                if ((int)lane >= o) { iM = max(uM + iS, iM); iS += uS; }
            }
            int64_t eS = __shfl_up_sync(0xffffffffu, iS, 1), eM = __shfl_up_sync(0xffffffffu, iM, 1);
            if (lane == 0) { eS = 0; eM = kNegInf; }
            int64_t Bl = max(B + eS, eM);                    // true busy-until entering this lane's chunk
            // re-serve the chunk
            bool idle_seen = false;
            for (uint32_t k = k0; k < k1; ++k) {
                const uint64_t i = cbase + in_pos[cbase + k];
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
                const int64_t issue = (int64_t)rec[1];
                const Served v = serve_terms(rs, mp, rec[0], issue, rec[2], q_ppm, div_q);
                const int64_t a = issue + (v.op ? v.xfer : 0);
                if (Bl <= a) idle_seen = true;
                Bl = max(a, Bl) + v.s;
                const int64_t done = Bl + (v.op ? 0 : v.xfer);
                const int64_t old = completion[i];
                if (done != old) { dstall += done - old; completion[i] = done; stall[i] = done - issue; max_c = max(max_c, (long long)done); }
            }
            served += __reduce_add_sync(0xffffffffu, k1 - k0);
            B = max(B + __shfl_sync(0xffffffffu, iS, 31), __shfl_sync(0xffffffffu, iM, 31));
            if (__any_sync(0xffffffffu, idle_seen)) break;   // the queue fell idle: the rest of the tile was served right
            if (served > kInLongBudget) { if (lane == 0) in_tile[tile].reserve = 1u; break; }
        }
        dstall = warp_sum(dstall);
        if (lane == 0 && dstall) atomicAdd((unsigned long long *)&in_tile[tile].fix_delta, (unsigned long long)dstall);
    }
    max_c = warp_max(max_c);
    if (lane == 0 && max_c != INT64_MIN) atomicMax(&ctrl->max_completion_ns, max_c);
}

// stall total of the batch: per tile the exact sum if it was re-served, else the as-if sum plus its corrections
__global__ void k_inorder_total(BatchCtrl *ctrl, const InTile *__restrict__ in_tile, uint32_t n_tiles) {
    if (ctrl->skip || ctrl->run_sort || !ctrl->inorder_used) return;
    long long tot = 0;
    for (uint32_t t = threadIdx.x; t < n_tiles; t += blockDim.x) {
        const InTile v = in_tile[t];
        tot += v.reserve ? v.true_sum : v.spec_sum + v.fix_delta;
    }
    tot = warp_sum(tot);
    if ((threadIdx.x & 31) == 0 && tot) atomicAdd((unsigned long long *)&ctrl->modeled_ns, (unsigned long long)tot);
}

uint64_t inorder_tile_records(uint64_t n, int sm_count) {
    const uint64_t want_tiles = std::min<uint64_t>(kInMaxTiles, (uint64_t)std::max(1, sm_count) * kInBlocksPerSM);   // one wave of resident blocks
    uint64_t t = (n + want_tiles - 1) / want_tiles;
    t = (t + kInChunk - 1) / kInChunk * kInChunk;
    return std::max<uint64_t>(t, kInChunk);
}

// dynamic shared memory of the serve kernel: two record buffers, counts, two position buffers, aggregates, per-die counters, head fill
size_t inorder_serve_smem(uint32_t n_dies) {
    return (size_t)2 * kInSlotBytes + kInCntBytes + 2 * kInPosBytes + (size_t)kInMaxQueues * 16 + (size_t)n_dies * 24 + kInMaxQueues;
}

static uint32_t inorder_row_stride(uint32_t n_queues) { return (n_queues + 1u + 7u) / 8u * 8u; }
size_t inorder_head_bytes(uint64_t tiles, uint32_t n_queues) { return tiles * n_queues * (size_t)kInHead * sizeof(InHead); }
size_t inorder_start_bytes(uint64_t n, uint32_t n_queues) {
    return ((n + kInChunk - 1) / kInChunk + 1) * (size_t)inorder_row_stride(n_queues) * sizeof(uint16_t);
}

cudaError_t launch_inorder(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    const uint64_t tile_records = inorder_tile_records(n, a.sm_count);
    const unsigned n_tiles = (unsigned)((n + tile_records - 1) / tile_records);
    const uint32_t R = a.mp.n_queues, nd = a.mp.n_dies, row_stride = inorder_row_stride(R);
    const size_t smem_serve = inorder_serve_smem(nd);
    static size_t set_serve = 0;
    if (smem_serve > set_serve) {
        cudaError_t e = cudaFuncSetAttribute(k_inorder_serve<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_serve);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(k_inorder_serve<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_serve);
        if (e != cudaSuccess) return e;
        set_serve = smem_serve;
    }
    InTile *tiles = reinterpret_cast<InTile *>(a.ws.in_tile);
    InHead *heads = reinterpret_cast<InHead *>(a.ws.in_head);
    cudaError_t em = cudaMemsetAsync(a.ws.in_list, 0, sizeof(uint32_t), st);
    if (em != cudaSuccess) return em;
    k_inorder_serve<false><<<n_tiles, kInThreads, smem_serve, st>>>(a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.status,
                                                                    a.ws.in_agg, a.ws.in_pos, a.ws.in_start, row_stride, a.stats_stage,
                                                                    a.completion, a.stall, a.ws.in_bin, tiles, heads, a.ws.in_headcnt);
    k_inorder_scan<<<(R + kInScanThreads - 1) / kInScanThreads, kInScanThreads, 0, st>>>(
        a.ctrl, a.mp_dev, n_tiles, a.ws.in_agg, a.ws.in_bin, a.busy, a.busy_stage, a.stats_stage, a.path == HBF_PATH_INORDER ? 1 : 0);
    const uint64_t fix_threads = (uint64_t)n_tiles * R;
    k_inorder_fixup<<<(unsigned)((fix_threads + kInFixThreads - 1) / kInFixThreads), kInFixThreads, 0, st>>>(
        R, n_tiles, a.ctrl, a.ws.in_bin, heads, a.ws.in_headcnt, a.completion, a.stall, tiles, a.ws.in_list);
    k_inorder_fixup_long<<<(unsigned)std::max(1, a.sm_count * 4), kInFixThreads, 0, st>>>(
        a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.ws.in_bin, a.ws.in_pos, a.ws.in_start, row_stride, a.completion, a.stall,
        tiles, a.ws.in_list);
    k_inorder_serve<true><<<n_tiles, kInThreads, smem_serve, st>>>(a.acc, n, tile_records, a.ranges, a.mp_dev, a.ctrl, a.status,
                                                                   a.ws.in_agg, a.ws.in_pos, a.ws.in_start, row_stride, a.stats_stage,
                                                                   a.completion, a.stall, a.ws.in_bin, tiles, heads, a.ws.in_headcnt);
    k_inorder_total<<<1, 256, 0, st>>>(a.ctrl, tiles, n_tiles);
    g_kernel_launches += 6;
    return cudaGetLastError();
}

}  // namespace hbf
