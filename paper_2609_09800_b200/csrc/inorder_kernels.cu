// In-order path of hbf_submit_batch: serves a batch whose records arrive in non-decreasing issue order
// without a global sort.  In such a batch the (issue, index) order of every queue is plain index order,
// so the batch is cut into contiguous tiles, one per resident thread block, that are served independently:
//   serve     every tile classifies and decodes its records, writes status[], counts, sums per-die bytes, and
//             serves its accesses AS IF every queue were idle when the tile begins; completions and stalls
//             are written as they are computed, in batch order.  Per queue it also keeps the composition
//             (S, M) of the maps B -> max(B + s, a + s) of its accesses (M is exactly the busy-until of the
//             as-if run) and the first few accesses of the queue in the tile (the head table);
//   scan      one thread per queue walks the tiles' aggregates in order: the true busy-until entering each
//             tile, and the final busy-until;
//   fix-up    one thread per (tile, queue) starts from the true entering busy-until and re-serves the head
//             table's accesses in order, until it meets an access that arrives when the queue is idle: from
//             there on the as-if run and the true run coincide (busy-until is monotone in its start value, so
//             the as-if run was idle there too);
//   straggle  a queue still backlogged past its head entries is re-served from the records: the tile's
//             block streams the tile again, keeps only that tile's straggling queues, and stops as soon as
//             each of them has fallen idle;
//   re-serve  a tile with many stragglers (the batch arrived on queues that were far behind) is served
//             again from the true entering busy-until, exactly.
// The serve pass is the only one that streams the whole batch: 24 B read and 16 B + 1 B written per access.
// Every global access of it is coalesced; nothing waits on another thread block, and no thread spins.
//
// Inside a tile the busy-until of every queue lives in shared memory.  The records are taken 32 at a time
// (a row per warp, rows dealt round-robin to the block's warps); all the per-record arithmetic runs in
// parallel, and only the read-serve-write of the queue state is done row after row, handed from warp to
// warp through the hardware's named barriers.  Records of one queue that fall into the same row are chained
// in registers with shuffles.
#include <algorithm>
#include <cstddef>
#include <type_traits>

#include "device_utils.cuh"

namespace hbf {

// Block shape of the serve kernel.  The per-queue state (32 KB) is all the shared memory a block needs, so
// several blocks share an SM, each with its own tile and its own row-after-row chain of queue updates.
#ifndef HBF_IN_THREADS
#define HBF_IN_THREADS 320
#endif
#ifndef HBF_IN_BLOCKS
#define HBF_IN_BLOCKS 2
#endif
constexpr int kInThreads = HBF_IN_THREADS;               // threads of a serve block
constexpr int kInBlocksPerSM = HBF_IN_BLOCKS;            // resident serve blocks per SM
constexpr int kInWarps = kInThreads / 32;
constexpr uint32_t kInTagStride = kInMaxQueues + 32;      // bytes of a warp's table of lane numbers: one per queue, one per lane
#ifndef HBF_IN_ROWS
#define HBF_IN_ROWS 2
#endif
#ifndef HBF_IN_PFDIST
#define HBF_IN_PFDIST 2
#endif
constexpr int kInPrefetchTurns = HBF_IN_PFDIST;          // how many of the warp's turns ahead its records are called into the L2
constexpr int kInRows = HBF_IN_ROWS;                     // rows of 32 records a warp serves per turn
static_assert(kInWarps >= 2 && kInWarps <= 15, "every warp owns one of the hardware barriers 1..15");

// One access, from its record: status, and for a modeled access its queue, die and service terms.
// (the in-order path is only chosen when every transfer time fits 31 bits)
struct Served { int st; uint32_t queue, die, op, xfer; int64_t s, cb; };
// long_service (here and below): set when one access's service time reaches 2^long_bits ns.  The serve pass keeps a tile's
// service-time sum per queue in 56 bits (55 and a sign); a tile has fewer than 2^22 records, so with every service below
// 2^33 ns (8.6 s) the sum cannot overflow; with retention on a claimed refresh quantum is added to a service, and both
// stay below 2^32.  A batch with a longer service is handed to the sort path like an unsorted one.
__device__ __forceinline__ Served serve_terms(const RangeSnap &rs, const ModelParams &mp, uint64_t addr, int64_t issue,
                                              uint64_t bf, int64_t q_ppm, const Div64 &div_q, unsigned &long_service, int long_bits) {
    Served r; r.queue = 0; r.die = 0; r.op = 0; r.s = 0; r.xfer = 0; r.cb = 0;
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    int g = 0;
    r.st = classify(rs, addr, issue, bytes, flags, &g);
    if (r.st == HBF_ST_READY) {
        const uint64_t off = rs.media_offset[g] + (addr - rs.base[g]);
        const Decoded d = decode(mp, off, bytes);
        r.op = flags & 1u;
        const Terms t = service_terms(mp, bytes, d.npages, r.op, q_ppm, div_q);
        r.queue = d.queue; r.die = d.die; r.s = t.s; r.xfer = (uint32_t)t.xfer; r.cb = t.cb;
        if ((uint64_t)t.s >> long_bits) long_service = 1u;
    }
    return r;
}

// The same terms for the common configuration (one registered range, power-of-two geometry, no thermal
// scaling in force, transfer table present): 32-bit arithmetic wherever the values allow it.
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
    r.xfer = cb <= (uint64_t)mp.xfer_tab_max_cb ? __ldg(mp.xfer_tab + (uint32_t)(cb >> mp.xfer_tab_shift))
                                                 : (uint32_t)div64(cb * 1000ull + mp.chan_bytes_per_us - 1ull, mp.div_chan);
    r.s = (int64_t)npages * (r.op ? mp.t_prog_ns : mp.t_read_ns);
    return r;
}
// The common configuration once more, laid out for the serve pass (a kernel argument: its fields are operands of the
// instructions that use them, which measured 1.8 % faster than seven 16-byte vectors in shared memory), every field a
// 32-bit operand where the values allow it (page times and the transfer table's reach below 2^32).
struct __align__(16) FastGeom {
    uint64_t base, length;                                  // the one registered range
    uint64_t media_offset; uint32_t perms, stripe_shift;
    uint32_t ch_mask, ch_shift, die_mask, chdie_shift;      // stripe unit -> channel, die, plane
    uint32_t plane_mask, dies, planes_q, plane_mask_q;      // planes_q = 1, plane_mask_q = 0 with one queue per die
    uint32_t page_mask, page_shift, gran_shift_read, gran_shift_prog;
    uint32_t tab_shift, tab_max_cb, t_read, t_prog;
    const uint32_t *xfer_tab; uint64_t pad;
};
// (the last condition: an access within the transfer table's reach spans few pages, and their unscaled service stays
// below 2^32 ns, so the common path needs no test of its own)
__device__ __forceinline__ bool fast_geom_ok(const FastRange &f, const ModelParams &mp) {
    const uint64_t pages = ((uint64_t)mp.xfer_tab_max_cb >> mp.page_shift) + 2ull;
    return f.on != 0u && mp.pow2_geom != 0u && mp.xfer_tab_max_cb != 0u && mp.t_read_ns < (1ll << 32) && mp.t_prog_ns < (1ll << 32) &&
           pages * (uint64_t)max(mp.t_read_ns, mp.t_prog_ns) < (1ull << 32);
}
__host__ __device__ __forceinline__ FastGeom make_fast_geom(const FastRange &f, const ModelParams &mp) {
    FastGeom g;
    g.base = f.base; g.length = f.length; g.media_offset = f.media_offset; g.perms = f.perms; g.stripe_shift = mp.stripe_shift;
    g.ch_mask = mp.channels - 1u; g.ch_shift = mp.ch_shift; g.die_mask = mp.dies - 1u; g.chdie_shift = mp.ch_shift + mp.die_shift;
    g.plane_mask = mp.planes - 1u; g.dies = mp.dies;
    g.planes_q = mp.queue_level == 0u ? mp.planes : 1u; g.plane_mask_q = mp.queue_level == 0u ? mp.planes - 1u : 0u;
    g.page_mask = (1u << mp.page_shift) - 1u; g.page_shift = mp.page_shift;
    g.gran_shift_read = mp.read_gran_shift; g.gran_shift_prog = mp.prog_gran_shift;
    g.tab_shift = mp.xfer_tab_shift; g.tab_max_cb = mp.xfer_tab_max_cb; g.t_read = (uint32_t)mp.t_read_ns; g.t_prog = (uint32_t)mp.t_prog_ns;
    g.xfer_tab = mp.xfer_tab; g.pad = 0;
    return g;
}
// No branches: every access computes every term, and the classification (the same tests in the same order as classify())
// only selects the status; the terms of an access that is not READY are never used.  (Early returns cost this pass
// about 47 instructions per row of 32 accesses, measured.)
__device__ __forceinline__ Served serve_terms_geom(const FastGeom &g, const ModelParams &mp, uint64_t addr, int64_t issue, uint64_t bf,
                                                  int64_t q_ppm, const Div64 &div_q, unsigned &long_service, int long_bits) {
    Served r;
    const uint32_t bytes = (uint32_t)bf, flags = (uint32_t)(bf >> 32);
    const uint64_t rel = addr - g.base;                       // wraps to a huge value below the base
    const uint32_t op = flags & 1u;
    const bool unsupported = bytes == 0u || flags > 1u || (uint32_t)((uint64_t)issue >> 32) >= (1u << (kIssueBits - 32));
    const bool outside = rel >= g.length;
    const bool partial = (uint64_t)bytes > g.length - rel;
    const bool denied = ((g.perms >> op) & 1u) == 0u;
    int st = denied ? HBF_ST_FAULT_PERM : HBF_ST_READY;
    st = partial ? HBF_ST_FAULT_PARTIAL : st;
    st = outside ? HBF_ST_NATIVE : st;
    r.st = unsupported ? HBF_ST_UNSUPPORTED : st;
    r.op = op;
    const uint64_t off = g.media_offset + rel;
    const uint32_t u = (uint32_t)(off >> g.stripe_shift);     // only the low interleave bits are used
    const uint32_t ch = u & g.ch_mask, di = (u >> g.ch_shift) & g.die_mask, pl = (u >> g.chdie_shift) & g.plane_mask_q;
    r.die = ch * g.dies + di;
    r.queue = r.die * g.planes_q + pl;
    const uint32_t npages = (uint32_t)(((uint64_t)((uint32_t)off & g.page_mask) + bytes + g.page_mask) >> g.page_shift);
    const uint32_t gs = op ? g.gran_shift_prog : g.gran_shift_read;
    const uint64_t gm = (1ull << gs) - 1ull;
    const uint64_t cb = ((uint64_t)bytes + gm) & ~gm;
    r.cb = (int64_t)cb;
    const uint64_t s0 = (uint64_t)npages * (op ? g.t_prog : g.t_read);
    if (cb <= (uint64_t)g.tab_max_cb) {
        r.xfer = __ldg(g.xfer_tab + ((uint32_t)cb >> g.tab_shift));
    } else {                                                  // a large access: rare
        r.xfer = (uint32_t)div64(cb * 1000ull + mp.chan_bytes_per_us - 1ull, mp.div_chan);
        if (s0 >> long_bits) long_service = 1u;
    }
    if (q_ppm == 1000000) {
        r.s = (int64_t)s0;
    } else {                                                  // thermal scaling in force: Eq. 3 (s0 < 2^50)
        r.s = (int64_t)div64(s0 * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);
        if ((uint64_t)r.s >> long_bits) long_service = 1u;
    }
    return r;
}
// The first kInHead accesses of every (tile, queue), as the serve pass saw them: all the fix-up needs in the common case.
// (Six, measured on the capacity stream at loads 0.3 to 0.9: eight cost 2.5 % more at every load for the table's traffic
// and bookkeeping and fell back to a second pass at the same load, between 0.6 and 0.7; five or fewer are faster still
// at low load but need the second pass from 0.6 on.)
constexpr int kInHead = 6;
struct InHead { int64_t m, s; uint32_t xo, idx; };       // arrival + service, service, transfer | op << 31, batch index
// Where entry ci of (tile, queue) sits: a tile's first entries side by side (the fix-up reads the first entry of every
// queue: one coalesced stretch instead of a record every 192 bytes), then every queue's later entries side by side (read
// only for the queues still behind, all of them at once).
__device__ __forceinline__ uint64_t head_slot(uint32_t tile, uint32_t R, uint32_t q, uint32_t ci) {
    const uint64_t base = (uint64_t)tile * R * kInHead;
    return ci == 0u ? base + q : base + R + (uint64_t)q * (kInHead - 1) + (ci - 1u);
}

// ======================================================================================================
// serve.  RESERVE = false: the streaming pass over every tile, every queue taken as idle at the tile's start.
// RESERVE = true: only for tiles the fix-up flagged (many queues stayed backlogged far into the tile): the
// same pass from the true entering busy-until, writing the exact results and nothing else.
//
// A tile is cut into rows of 32 consecutive records; warp w takes rows w, w + W, w + 2W, ...  Everything that
// does not depend on the queues' state (load, classification, decode, service terms, the ranking of lanes that
// hold the same queue) happens in parallel.  The queue update itself (read the busy-until, serve, write it
// back: a handful of instructions) is done row after row: the warp of row r waits on a hardware barrier that
// the warp of row r - 1 arrives at when its update is in shared memory.  Warp w owns barrier 1 + w: it is the
// only one that waits on it, and warp w - 1 the only one that arrives, so uses of a barrier cannot overlap.
// ======================================================================================================
// The extra operands are not used by the instruction: naming them makes the compiler finish computing them
// before the wait instead of after it.  The aligned forms of the barrier instructions are used (measured a
// little faster): like __syncthreads(), they sit where the warp's control flow is uniform.
__device__ __forceinline__ void row_wait(int id, int64_t m, long long s8, const void *pq, uint32_t pc, bool last) {
    asm volatile("barrier.cta.sync.aligned %0, 64;" ::"r"(id), "l"(m), "l"(s8), "l"(pq), "r"(pc), "r"((int)last) : "memory");
}
__device__ __forceinline__ void row_pass(int id) { asm volatile("barrier.cta.arrive.aligned %0, 64;" ::"r"(id) : "memory"); }

__device__ __forceinline__ void row_wait2(int id, int64_t m, long long s8, const void *pq, uint32_t pc, bool last,
                                          int64_t m2, long long s82, const void *pq2, uint32_t pc2, bool last2) {
    asm volatile("barrier.cta.sync.aligned %0, 64;" ::"r"(id), "l"(m), "l"(s8), "l"(pq), "r"(pc), "r"((int)last),
                 "l"(m2), "l"(s82), "l"(pq2), "r"(pc2), "r"((int)last2) : "memory");
}

// DEBT = true (retention on): a modeled access with a batch index below the claim limit pays one refresh quantum (a page
// read and a page program, scaled like any service, Eq. 3) before its own service; the streaming pass counts the
// claims per die.
template <bool RESERVE, bool DEBT>
__global__ void __launch_bounds__(kInThreads, kInBlocksPerSM)
k_inorder_serve(const hbf_access_t *__restrict__ acc, uint64_t n, const __grid_constant__ InTileMap tmap, const RangeSnap *__restrict__ ranges_g,
                const __grid_constant__ ModelParams mp_arg, const __grid_constant__ FastRange fast_arg, BatchCtrl *ctrl, uint8_t *__restrict__ status, int64_t *__restrict__ in_agg,
                hbf_die_stats_t *stats_stage, int64_t *__restrict__ completion, int64_t *__restrict__ stall,
                const int64_t *__restrict__ in_bin, InTile *in_tile, InHead *__restrict__ in_head, uint8_t *__restrict__ in_headcnt,
                const int64_t *__restrict__ busy, const unsigned long long *claim_limit_p, uint32_t *die_claims,
                const __grid_constant__ RetDev ret, uint16_t *__restrict__ in_qid, uint32_t qid_stride,
                TileBalance *bal, uint32_t bal_seq, const __grid_constant__ FastGeom geom, const uint32_t head_depth) {
    extern __shared__ __align__(16) unsigned char in_smem[];
    __shared__ long long s_red[2];
    __shared__ unsigned long long s_t0;                   // when this block took its tile (0: its time is not recorded)
    __shared__ uint32_t s_heads_full;                     // queues whose head entries are complete
    __shared__ ModelParams mp;                            // measured: reads from shared memory beat reads of the argument
    __shared__ FastRange fast_range;

    if (ctrl->skip || ctrl->run_sort) return;             // (run_sort set this early: the batch went to the sort path at its start)
    if (RESERVE && (!ctrl->inorder_used || !in_tile[blockIdx.x].reserve)) return;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const RangeSnap &rs = *ranges_g;                      // read through the cache; the common configuration does not touch it
    if (tid == 0) { mp = mp_arg; fast_range = fast_arg; }
    if (DEBT && !RESERVE && tid == 0 && blockIdx.x == 0) ret.st->observed_inline = 1u;
    if (!RESERVE && bal && tid == 0 && blockIdx.x == 0) { bal->strag_seq = bal_seq; bal->strag_max = 0u; bal->strag_flagged = 0u; bal->strag_depth = head_depth; }
    const uint32_t R = mp_arg.n_queues, n_dies = mp_arg.n_dies;
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    // one range, power-of-two geometry, transfer table, no thermal scaling in force: the short form of the terms
    const bool fast_on = fast_geom_ok(fast_arg, mp_arg);
    const uint32_t ret_row_shift = mp_arg.ch_shift + mp_arg.die_shift + mp_arg.plane_shift;   // stripe unit -> row of stripe units on its plane
    const uint64_t claim_limit = DEBT ? *claim_limit_p : 0ull;
    const int64_t quantum_ns = !DEBT ? 0 : q_ppm == 1000000 ? mp_arg.t_read_ns + mp_arg.t_prog_ns
        : (int64_t)div64((uint64_t)(mp_arg.t_read_ns + mp_arg.t_prog_ns) * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);

    // [queues] x: busy-until of the run in progress; y: service time served in this tile << 8 | head-table entries written
    longlong2 *qst = reinterpret_cast<longlong2 *>(in_smem);
    uint32_t *st_br_lo = reinterpret_cast<uint32_t *>(qst + kInMaxQueues), *st_br_hi = st_br_lo + n_dies;   // per die
    uint32_t *st_bp_lo = st_br_hi + n_dies, *st_bp_hi = st_bp_lo + n_dies;
    uint32_t *st_nr = st_bp_hi + n_dies, *st_np = st_nr + n_dies;
    uint32_t *st_claims = st_np + n_dies;                 // refresh quanta claimed on each die (claims variant)
    // per warp and row of a turn: a byte per queue (which lane of the row holds it) and one per lane
    uint8_t *warp_tag = reinterpret_cast<uint8_t *>(st_claims + n_dies) + (uint32_t)(threadIdx.x >> 5) * (kInRows * kInTagStride);

    // Which tile this block serves.  Two blocks share an SM, and the hardware favours the one in the lower warp slots: with
    // equal tiles it finishes about 12 % earlier (measured) and the pass lasts as long as the other one.  So the tiles come in
    // two sizes; a block reads off its warp slot which kind of block it is and takes the next tile of the matching size (or,
    // should one size run out, of the other: every tile is handed out exactly once whatever the slots say).
    __shared__ uint32_t s_tile_id;
    if (!RESERVE) {
        if (tid == 0) {
            uint32_t t = blockIdx.x;
            unsigned long long t0 = 0ull;
            if (tmap.n_big != 0u) {
                unsigned slot;
                asm volatile("mov.u32 %0, %%warpid;" : "=r"(slot));
                const uint32_t late = slot >= 4u ? 1u : 0u;   // warp 0 of the block that came second sits past the first four slots
                if (bal) {
                    // the tile of this SM and this kind; should it be gone (the slots did not say what they usually say),
                    // any tile that is left: every tile is taken exactly once, marked with the batch's number
                    unsigned sm;
                    asm volatile("mov.u32 %0, %%smid;" : "=r"(sm));
                    const uint32_t want = late * tmap.n_big + sm;
                    bool mine = sm < tmap.n_big && atomicExch(&bal->claim[want], bal_seq) != bal_seq;
                    t = want;
                    for (uint32_t k = 0; !mine && k < tmap.n_tiles; ++k) { t = k; mine = atomicExch(&bal->claim[k], bal_seq) != bal_seq; }
                    if (t == want) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
                } else {
                    const uint32_t have[2] = {tmap.n_big, tmap.n_tiles - tmap.n_big};
                    uint32_t k = atomicAdd(&ctrl->role_count[late], 1u);
                    if (k < have[late]) t = late ? tmap.n_big + k : k;
                    else { k = atomicAdd(&ctrl->role_count[1u - late], 1u); t = late ? k : tmap.n_big + k; }
                }
            }
            s_tile_id = t; s_t0 = t0;
        }
        __syncthreads();
    }
    const uint32_t tile = RESERVE ? blockIdx.x : s_tile_id;
    const uint64_t tile_begin = tile_first(tmap, tile);
    const uint64_t tile_end = tile_last(tmap, tile);

    for (uint32_t i = tid; i < kInMaxQueues; i += kInThreads) qst[i] = make_longlong2(kNegInf, 0);
    if (RESERVE) {
        __syncthreads();
        for (uint32_t q = tid; q < R; q += kInThreads) qst[q].x = in_bin[(uint64_t)blockIdx.x * R + q];
    } else {
        for (uint32_t d = tid; d < n_dies * 7u; d += kInThreads) st_br_lo[d] = 0u;
        if (tile == 0u) {                                    // the first tile knows its entering state: it is served exactly
            __syncthreads();
            for (uint32_t q = tid; q < R; q += kInThreads) qst[q].x = busy[q];
        }
    }
    uint32_t c_native = 0, c_ready = 0, c_valid = 0;         // per thread: far below 2^32 (a batch is below 2^30 records)
    unsigned c_unsorted = (DEBT && ((uint64_t)quantum_ns >> 32)) ? 1u : 0u;   // (or a service, or a refresh quantum, of 2^32 ns or more)
    long long sum_stall = 0, max_c = INT64_MIN;

    if (tid < 2) s_red[tid] = tid == 1 ? INT64_MIN : 0;
    if (tid == 0) s_heads_full = 0u;
    __syncthreads();

    // A warp's turn covers kInRows consecutive rows: their arithmetic interleaves, and their queue updates
    // follow one another inside one wait/pass pair.
    constexpr int K = kInRows;
    // inside a tile everything is indexed by 32-bit offsets from the tile's first record (a batch is below 2^30 records)
    const uint32_t tile_len = tile_end > tile_begin ? (uint32_t)(tile_end - tile_begin) : 0u;
    const hbf_access_t *acc_t = acc + tile_begin;
    int64_t *completion_t = completion + tile_begin, *stall_t = stall + tile_begin;
    uint8_t *status_t = status ? status + tile_begin : nullptr;
    uint16_t *qid_t = in_qid + (uint64_t)tile * qid_stride;   // the straggle pass filters the head of the tile by these
    const uint32_t rows = (tile_len + 31u) / 32u;
    const uint32_t turns = (rows + K - 1) / K;
    const unsigned le_mask = lanemask_lt() | (1u << lane);
    const int my_bar = 1 + warp, next_bar = 1 + (warp + 1 == kInWarps ? 0 : warp + 1);

    // the records of the warp's next turn are already on their way while this one is served
    uint64_t nx_addr[K], nx_issue[K], nx_bf[K];
    int64_t nx_prev[K];                                      // issue time of the record before the lane's own (same cache line, mostly)
#pragma unroll
    for (int u = 0; u < K; ++u) { nx_addr[u] = 0; nx_issue[u] = 0; nx_bf[u] = 0; nx_prev[u] = INT64_MIN; }
    const bool first_tile = tile_begin == 0;
    const bool pf_lane = lane < 24;
    const char *pf_base = reinterpret_cast<const char *>(acc_t) + lane * 32;
    auto fetch = [&](uint32_t turn) {
#pragma unroll
        for (int u = 0; u < K; ++u) {
            const uint32_t j = (turn * K + u) * 32u + (uint32_t)lane;
            if (j < tile_len) {
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc_t + j);
                nx_addr[u] = __ldcs(rec); nx_issue[u] = __ldcs(rec + 1); nx_bf[u] = __ldcs(rec + 2);   // read once: streaming loads
                if (!RESERVE) nx_prev[u] = (j > 0u || !first_tile) ? (int64_t)__ldg(rec - 2) : INT64_MIN;
            }
        }
    };
    fetch((uint32_t)warp);

    // A turn whose rows are all complete (every turn but the last of a batch whose size is not a multiple of 32) runs
    // a copy of the code that has no bounds tests.
    for (uint32_t turn = (uint32_t)warp; turn < turns; turn += kInWarps) {
      auto whole_turn = [&](auto full_tag) {
        constexpr bool FULL = decltype(full_tag)::value;
        uint32_t i[K];                                       // offsets from the tile's first record
        bool valid[K], ready[K], last[K];
        int64_t issue[K], a[K], S[K], M[K], B[K];
        Served v[K];
        uint32_t rank1[K], pc[K], c0[K], c1[K], qi[K];
        longlong2 *pq[K];
        int64_t prev[K];
        uint64_t addr[K], bf[K];
#pragma unroll
        for (int u = 0; u < K; ++u) {
            i[u] = (turn * K + u) * 32u + (uint32_t)lane;
            valid[u] = FULL || i[u] < tile_len;
            addr[u] = nx_addr[u]; bf[u] = nx_bf[u]; issue[u] = (int64_t)nx_issue[u]; prev[u] = nx_prev[u];
        }
        fetch(turn + kInWarps);
        {                                                    // and the turn after that is called into the L2
            const uint32_t first = (turn + kInPrefetchTurns * kInWarps) * (uint32_t)(K * 32);
            if (pf_lane && first + K * 32 <= tile_len) {     // 24 lanes cover a row's 768 bytes in 32-byte sectors
                const char *p = pf_base + (size_t)first * sizeof(hbf_access_t);
#pragma unroll
                for (int u = 0; u < K; ++u) asm volatile("prefetch.global.L2 [%0];" ::"l"(p + u * 768));
            }
        }
        // ---- terms ---------------------------------------------------------------------------------------
#pragma unroll
        for (int u = 0; u < K; ++u) {
            v[u].st = HBF_ST_NATIVE; v[u].queue = 0; v[u].die = 0; v[u].op = 0; v[u].s = 0; v[u].xfer = 0; v[u].cb = 0;
            if (valid[u])
                v[u] = fast_on ? serve_terms_geom(geom, mp, addr[u], issue[u], bf[u], q_ppm, div_q, c_unsorted, DEBT ? 32 : 33)
                                 : serve_terms(rs, mp, addr[u], issue[u], bf[u], q_ppm, div_q, c_unsorted, DEBT ? 32 : 33);
            ready[u] = valid[u] && v[u].st == HBF_ST_READY;
            if (DEBT && ready[u] && tile_begin + i[u] < claim_limit) {
                v[u].s += quantum_ns;
                if (!RESERVE) atomicAdd(&st_claims[v[u].die], 1u);
            }
            if (DEBT && !RESERVE && ready[u] && !v[u].op) {  // read disturb: the read's pages, on the block of its first page
                if (fast_on && ret.pow2 != 0u) {
                    // one range, powers of two all the way down: the block from shifts and masks (the general form below
                    // divides twice; it took the pass from 2.0 to 2.9 ms)
                    const uint64_t off = geom.media_offset + (addr[u] - geom.base);
                    const uint32_t npages = (uint32_t)(((uint64_t)((uint32_t)off & geom.page_mask) + (uint32_t)bf[u] + geom.page_mask) >> geom.page_shift);
                    const uint32_t row = (uint32_t)((off >> geom.stripe_shift) >> ret_row_shift);     // (the wrap of the general form too: the block inside the plane)
                    const uint32_t in_stripe = ((uint32_t)off & ((1u << geom.stripe_shift) - 1u)) >> geom.page_shift;
                    const uint32_t blk = ((row << mp_arg.pages_per_stripe_shift) + in_stripe) >> ret.ppb_shift;
                    const uint32_t pl = (uint32_t)(off >> (geom.stripe_shift + geom.chdie_shift)) & geom.plane_mask;
                    atomicAdd(&ret.disturb[((v[u].die << mp_arg.plane_shift) + pl) * ret.bpp + (blk & (ret.bpp - 1u))], npages);
                } else {
                    uint64_t off;
                    if (fast_on) off = fast_range.media_offset + (addr[u] - fast_range.base);
                    else { int g = 0; classify(rs, addr[u], issue[u], (uint32_t)bf[u], (uint32_t)(bf[u] >> 32), &g); off = rs.media_offset[g] + (addr[u] - rs.base[g]); }
                    const uint32_t page_mask = (1u << mp.page_shift) - 1u;
                    const uint32_t npages = (uint32_t)(((uint64_t)((uint32_t)off & page_mask) + (uint32_t)bf[u] + page_mask) >> mp.page_shift);
                    atomicAdd(&ret.disturb[ret_block_of(mp, ret, off)], npages);
                }
            }
        }
        // ---- which lanes of a row hold the same queue: every lane writes its number where its queue's entry is in the
        // warp's own table and reads the entry back (the answer is needed only further down: the latency is covered).
        // Nothing is ever cleared: a lane reads what a lane of this row wrote.  Accesses that are not modeled have an
        // entry per lane.  (`match_any` for every row kept the unit that executes it busy three quarters of the time.)
        uint8_t *tag_at[K];
        uint32_t tagged[K];
#pragma unroll
        for (int u = 0; u < K; ++u) { tag_at[u] = warp_tag + u * kInTagStride + (ready[u] ? v[u].queue : kInMaxQueues + (uint32_t)lane); *tag_at[u] = (uint8_t)lane; }
        __syncwarp();
#pragma unroll
        for (int u = 0; u < K; ++u) tagged[u] = *reinterpret_cast<volatile uint8_t *>(tag_at[u]);
        if (!RESERVE && turn * (uint32_t)(K * 32) < qid_stride) {   // (the stride is a multiple of a turn's records)
#pragma unroll
            for (int u = 0; u < K; ++u)
                if (valid[u]) qid_t[i[u]] = ready[u] ? (uint16_t)v[u].queue : (uint16_t)kInMaxQueues;   // (one past the last queue: not modeled)
        }
        if (!RESERVE) {
#pragma unroll
            for (int u = 0; u < K; ++u) {
                if (valid[u]) {
                    c_unsorted |= issue[u] < prev[u] ? 1u : 0u;
                    if (status_t) status_t[i[u]] = (uint8_t)v[u].st;
                    c_valid += 1u;
                    c_ready += ready[u] ? 1u : 0u;
                    c_native += v[u].st == HBF_ST_NATIVE ? 1u : 0u;
                    if (ready[u]) {
                        // charged bytes < 2^33: add the low word, carry into the high word when it wraps (a form that counts
                        // granules in one word and sends oversized accesses to the 64-bit totals measured slower)
                        const uint32_t lo = (uint32_t)v[u].cb, hi = (uint32_t)((uint64_t)v[u].cb >> 32);
                        uint32_t *plo = v[u].op ? st_bp_lo : st_br_lo, *phi = v[u].op ? st_bp_hi : st_br_hi;
                        atomicAdd(v[u].op ? &st_np[v[u].die] : &st_nr[v[u].die], 1u);
                        const uint32_t old = atomicAdd(&plo[v[u].die], lo);
                        const uint32_t carry = hi + ((old + lo) < old ? 1u : 0u);
                        if (carry) atomicAdd(&phi[v[u].die], carry);
                    }
                }
            }
        }
        // The rest of the turn exists twice: with the head-table bookkeeping, and without it once every queue of the
        // tile has its head entries (after a few percent of a large tile).  The flag is the same for the whole warp.
        const bool heads_on = !RESERVE && *reinterpret_cast<volatile uint32_t *>(&s_heads_full) < R;
        auto rest_of_turn = [&](auto heads_tag) {
        constexpr bool HEADS = decltype(heads_tag)::value;
        // ---- per row: the accesses of a lane's queue, up to the lane's own, as one map B -> max(B + S, M), composed
        // in lane order, so that the ordered part below is one application of it whatever the row holds
#pragma unroll
        for (int u = 0; u < K; ++u) {
            a[u] = issue[u] + (int64_t)(v[u].op ? v[u].xfer : 0u);   // arrival at the queue: a program's data is transferred first
            rank1[u] = 1u;                                  // this access is the rank1-th of its queue in the row
            last[u] = ready[u];                             // no later access of this queue in the row
            pc[u] = HEADS ? 1u : 0u;                        // accesses of this queue in the row
            S[u] = v[u].s; M[u] = a[u] + v[u].s;
            // A lane that did not read its own number back shares its queue with another lane of the row: one row in five.
            const bool loser = tagged[u] != (uint32_t)lane;
            if (__any_sync(0xffffffffu, loser)) {
                // Second round: the lanes that lost write again.  In a pair the winner now reads its peer's number and the
                // loser its own; a loser that loses again has two peers or more, and only then is the row matched in full.
                if (loser) *tag_at[u] = (uint8_t)lane;
                __syncwarp();
                const uint32_t t2 = *reinterpret_cast<volatile uint8_t *>(tag_at[u]);
                if (!__any_sync(0xffffffffu, loser && t2 != (uint32_t)lane)) {
                    // pairs only (nearly always): the second lane of a pair composes its peer's map with its own
                    const uint32_t peer = loser ? tagged[u] : t2;                  // the lane itself when it has none
                    const bool second = peer < (uint32_t)lane;
                    const int64_t mp_ = __shfl_sync(0xffffffffu, M[u], (int)peer), sp_ = __shfl_sync(0xffffffffu, (int64_t)v[u].s, (int)peer);
                    if (second) { M[u] = max(mp_, a[u]) + v[u].s; S[u] = sp_ + v[u].s; rank1[u] = 2u; }
                    if (peer > (uint32_t)lane) last[u] = false;
                    if (HEADS && peer != (uint32_t)lane) pc[u] = 2u;
                } else {
                    const unsigned peers = __match_any_sync(0xffffffffu, ready[u] ? v[u].queue : (0x10000u | (uint32_t)lane));
                    const unsigned le = peers & le_mask;
                    rank1[u] = (uint32_t)__popc(le);
                    last[u] = ready[u] && (peers >> lane) == 1u;
                    pc[u] = HEADS ? (uint32_t)__popc(peers) : 0u;
                    // Every lane composes the maps of the lanes of its queue up to its own by doubling: it holds the map of a
                    // stretch of them that ends with itself and the lane before that stretch, takes that lane's stretch in front
                    // of its own, and goes on from the lane before that one; ceil(log2(most lanes on one queue)) rounds.
                    // (One lane after the other took as many rounds as lanes: 12.7 warp instructions per part where the parts
                    // of a split access, neighbours on one queue, fill the rows, against 9 per access unsplit.)
                    const unsigned before = le & ~(1u << lane);
                    int prev = before ? 31 - __clz((int)before) : -1;
                    const uint32_t n_max = __reduce_max_sync(0xffffffffu, rank1[u]);
                    for (uint32_t span = 1; span < n_max; span <<= 1) {
                        const int src = prev >= 0 ? prev : lane;
                        const int64_t Se = __shfl_sync(0xffffffffu, S[u], src), Me = __shfl_sync(0xffffffffu, M[u], src);
                        const int pe = __shfl_sync(0xffffffffu, prev, src);
                        if (prev >= 0) { M[u] = max((int64_t)(Me + S[u]), M[u]); S[u] = Se + S[u]; prev = pe; }
                    }
                }
            }
            qi[u] = ready[u] ? v[u].queue : 0u;
            pq[u] = qst + qi[u];
        }
        // ---- the queue updates, in row order: everything they need is in registers before the wait ---------------
        if (turn > 0) {
            if (K == 1) row_wait(my_bar, M[0], S[0], pq[0], pc[0], last[0]);
            else row_wait2(my_bar, M[0], S[0], pq[0], pc[0], last[0], M[K - 1], S[K - 1], pq[K - 1], pc[K - 1], last[K - 1]);
        }
#pragma unroll
        for (int u = 0; u < K; ++u) {
            const longlong2 state = *pq[u];
            B[u] = max((int64_t)(state.x + S[u]), M[u]);
            uint32_t inc = 0u;
            if (HEADS) {
                c0[u] = min((uint32_t)state.y & 0xffu, head_depth);
                inc = min(pc[u], head_depth - c0[u]);
                c1[u] = c0[u] + inc;
            }
            if (last[u]) *pq[u] = make_longlong2(B[u], state.y + (S[u] << 8) + (long long)inc);
            if (u + 1 < K) __syncwarp();                     // the next row may hold the same queues
        }
        if (turn + 1 < turns) row_pass(next_bar);
        // ---- results ---------------------------------------------------------------------------------------
#pragma unroll
        for (int u = 0; u < K; ++u) {
            if (valid[u]) {
                const int64_t done = ready[u] ? B[u] + (int64_t)(v[u].op ? 0u : v[u].xfer) : issue[u];   // a read's data is transferred after its service;
                const int64_t st = done - issue[u];                                                    // not modeled: completion = issue, no stall
                sum_stall += st; max_c = max(max_c, ready[u] ? (long long)done : (long long)INT64_MIN);
                if (HEADS && ready[u]) {
                    const uint32_t ci = c0[u] + rank1[u] - 1u;
                    if (ci < head_depth) {
                        InHead h; h.m = a[u] + v[u].s; h.s = v[u].s; h.xo = v[u].xfer | (v[u].op << 31); h.idx = (uint32_t)tile_begin + i[u];
                        in_head[head_slot(tile, R, qi[u], ci)] = h;
                    }
                    if (last[u] && c1[u] != c0[u] && c1[u] == head_depth) atomicAdd(&s_heads_full, 1u);
                }
                // results are written once and not read again by this pass: streaming stores
                __stcs(reinterpret_cast<long long *>(completion_t + i[u]), (long long)done);
                __stcs(reinterpret_cast<long long *>(stall_t + i[u]), (long long)st);
            }
        }
        };
        if (heads_on) rest_of_turn(std::true_type{}); else rest_of_turn(std::false_type{});
      };
      if ((turn * K + K) * 32u <= tile_len) whole_turn(std::true_type{}); else whole_turn(std::false_type{});
    }

    __syncthreads();
    if (!RESERVE) {
        longlong2 *out = reinterpret_cast<longlong2 *>(in_agg) + (uint64_t)tile * R;
        for (uint32_t q = tid; q < R; q += kInThreads) {
            const longlong2 v = qst[q];
            out[q] = make_longlong2(v.y >> 8, v.x);
            in_headcnt[(uint64_t)tile * R + q] = (uint8_t)(v.y & 0xff);
        }
        for (uint32_t d = tid; d < n_dies; d += kInThreads) {
            unsigned long long *g = reinterpret_cast<unsigned long long *>(stats_stage + d);
            const unsigned long long br = ((unsigned long long)st_br_hi[d] << 32) | st_br_lo[d];
            const unsigned long long bp = ((unsigned long long)st_bp_hi[d] << 32) | st_bp_lo[d];
            if (br) atomicAdd(&g[1], br);
            if (bp) atomicAdd(&g[2], bp);
            if (st_nr[d]) atomicAdd(&g[4], (unsigned long long)st_nr[d]);
            if (st_np[d]) atomicAdd(&g[5], (unsigned long long)st_np[d]);
            if (DEBT && st_claims[d]) atomicAdd(&die_claims[d], st_claims[d]);
        }
        const unsigned long long w_native = (unsigned long long)warp_sum((long long)c_native);
        const unsigned long long w_ready = (unsigned long long)warp_sum((long long)c_ready);
        const unsigned long long w_fault = (unsigned long long)warp_sum((long long)(c_valid - c_ready - c_native));   // every other status is a fault
        c_unsorted = __any_sync(0xffffffffu, c_unsorted);
        if (lane == 0) {
            if (w_native) atomicAdd(&ctrl->n_native, w_native);
            if (w_ready) atomicAdd(&ctrl->n_ready, w_ready);
            if (w_fault) atomicAdd(&ctrl->n_fault, w_fault);
            if (c_unsorted) atomicOr(&ctrl->unsorted, 1u);
        }
    }
    sum_stall = warp_sum(sum_stall); max_c = warp_max(max_c);
    if (lane == 0) { atomicAdd((unsigned long long *)&s_red[0], (unsigned long long)sum_stall); atomicMax(&s_red[1], max_c); }
    __syncthreads();
    if (tid == 0) {
        if (RESERVE) in_tile[tile].true_sum = s_red[0];
        else { InTile t; t.spec_sum = s_red[0]; t.fix_delta = 0; t.true_sum = 0; t.reserve = 0u; t.stragglers = 0u; in_tile[tile] = t; }
        if (s_red[1] != INT64_MIN) atomicMax(&ctrl->max_completion_ns, s_red[1]);
        if (!RESERVE && bal) {                               // how many records, how long: what the next batches' tile sizes follow from
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            bal->len[tile] = tile_len;
            bal->ns[tile] = s_t0 ? (uint32_t)min(now - s_t0, 0xffffffffull) : 0u;
        }
    }
}

// ======================================================================================================
// scan over tiles; also decides what happens to the batch.
// A block takes kInScanQueues consecutive queues (threadIdx.x) and cuts the tiles into kInScanChunks runs of
// consecutive tiles (threadIdx.y).  Every thread composes the aggregates (S, M) of its run, the runs' maps are
// composed in order through shared memory, and the thread walks its run again from the true busy-until entering
// it, which it stores for every tile.  The kInScanQueues lanes of a run read consecutive 16-byte aggregates:
// whole 128-byte lines.  A few tiles per thread and all blocks resident at once: no long chain of loads.
// ======================================================================================================
constexpr int kInScanChunks = 64;
constexpr int kInScanQueues = 8;

__global__ void __launch_bounds__(kInScanQueues * kInScanChunks)
k_inorder_scan(BatchCtrl *ctrl, const ModelParams *__restrict__ mp, uint32_t n_tiles, const int64_t *__restrict__ in_agg,
               int64_t *__restrict__ in_bin, const int64_t *__restrict__ busy, int64_t *__restrict__ busy_stage,
               hbf_die_stats_t *stats_stage, int forced) {
    __shared__ longlong2 s_map[kInScanChunks][kInScanQueues];
    if (ctrl->skip || ctrl->run_sort) return;
    const bool fault = ctrl->n_fault != 0, unsorted = ctrl->unsorted != 0u;   // settled by the serve pass: every thread sees the same
    if (blockIdx.x == 0 && threadIdx.x == 0 && threadIdx.y == 0) {
        if (fault) { ctrl->code = HBF_E_ACCESS_FAULT; ctrl->skip = 1; }                 // fail closed: refuse the batch
        else if (unsorted && forced) { ctrl->code = HBF_E_INVAL; ctrl->skip = 1; }
        else if (unsorted) ctrl->run_sort = 1u;                                         // hand the batch to the sort path
        else ctrl->inorder_used = 1u;
    }
    if (fault || unsorted) return;
    const uint32_t R = mp->n_queues;
    const uint32_t r = blockIdx.x * (uint32_t)kInScanQueues + threadIdx.x, chunk = threadIdx.y;
    const uint32_t per = (n_tiles + kInScanChunks - 1) / kInScanChunks;
    const uint32_t t_lo = min(n_tiles, chunk * per), t_hi = min(n_tiles, t_lo + per);
    const bool live = r < R;
    const longlong2 *agg = reinterpret_cast<const longlong2 *>(in_agg) + r;
    long long S = 0, M = kNegInf;                            // the run's own map
    if (live) {
        for (uint32_t t = t_lo; t < t_hi; ++t) {
            const longlong2 v = agg[(uint64_t)t * R];
            M = max((int64_t)(M + v.x), (int64_t)v.y); S += v.x;
        }
    }
    s_map[chunk][threadIdx.x] = make_longlong2(S, M);
    __syncthreads();
    long long tot = 0;
    if (live) {
        // busy-until entering the run: the state earlier batches left, through the maps of the runs before it
        int64_t B = busy[r];
        for (uint32_t c = 0; c < chunk; ++c) { const longlong2 v = s_map[c][threadIdx.x]; B = max((int64_t)(B + v.x), (int64_t)v.y); }
        for (uint32_t t = t_lo; t < t_hi; ++t) {
            const longlong2 v = agg[(uint64_t)t * R];
            in_bin[(uint64_t)t * R + r] = B;
            B = max((int64_t)(B + v.x), (int64_t)v.y);
        }
        if (chunk == kInScanChunks - 1) {                    // the last run ends at the batch's end (empty runs pass B through)
            busy_stage[r] = B;
            for (uint32_t c = 0; c < (uint32_t)kInScanChunks; ++c) tot += s_map[c][threadIdx.x].x;
            const uint32_t die = mp->queue_level == 0u ? r / mp->planes : r;
            if (tot) atomicAdd(reinterpret_cast<unsigned long long *>(&stats_stage[die].busy_ns), (unsigned long long)tot);
        }
    }
    tot = warp_sum(tot);                                     // (only the last run's threads carry a total)
    if (((threadIdx.y * kInScanQueues + threadIdx.x) & 31u) == 0u && tot)
        atomicAdd((unsigned long long *)&ctrl->service_ns, (unsigned long long)tot);
}

// Queue of an access of the common configuration (one range, power-of-two geometry), or ~0 when the address
// lies outside the range.  In a batch that was not refused every access inside the range is modeled.
__device__ __forceinline__ uint32_t fast_queue(const FastRange &f, const ModelParams &mp, uint64_t addr) {
    const uint64_t rel = addr - f.base;
    if (rel >= f.length) return 0xffffffffu;
    const uint32_t u = (uint32_t)((f.media_offset + rel) >> mp.stripe_shift);
    const uint32_t ch = u & (mp.channels - 1u), di = (u >> mp.ch_shift) & (mp.dies - 1u);
    const uint32_t pl = (u >> (mp.ch_shift + mp.die_shift)) & (mp.planes - 1u);
    const uint32_t die = ch * mp.dies + di;
    return mp.queue_level == 0u ? die * mp.planes + pl : die;
}

// ======================================================================================================
// fix-up and straggle: one block per tile.
// Fix-up.  The true run differs from the as-if-idle run only at the head of each (tile, queue): a thread starts
// from the true entering busy-until of its queues and re-serves the head table's accesses in order, until it meets
// one that arrives on an idle queue; from there on the as-if run was right.  The head entries of a (tile, queue) are
// contiguous, so they are fetched in two rounds (the first two, which settle nearly every queue, then the rest at
// once) instead of one dependent load per entry.  A queue still backlogged after kInHead accesses is a straggler;
// a tile with many of them (the batch arrived on queues that were far behind) is flagged to be served again whole.
// Straggle.  The block streams the head of the tile again, keeps the modeled records of the straggling queues in
// batch order and re-serves them a chunk at a time, carrying both the true run (from the true entering
// busy-until) and the as-if-idle run (to know what the serve pass wrote).  A queue is done when the two runs meet:
// from there on the serve pass was right.  The block stops at the chunk in which its last queue is done.
// What it streams: for the first kInQidPrefix records of every tile the serve pass left the queue of each record
// as a 16-bit number (kInMaxQueues: not modeled), so the filter reads 2 bytes per record, 32 records per thread and turn;
// past that prefix (queues that stay backlogged for very long) it decodes the queue from the records.
// ======================================================================================================
// The general form of the terms (several ranges, any geometry, thermal scaling), kept out of line here: this kernel runs
// nearly straight through once per block, so what it costs is fetching its instructions, and the common configuration
// never takes this path.
__device__ __noinline__ Served serve_terms_general(const RangeSnap &rs, const ModelParams &mp, uint64_t addr, int64_t issue, uint64_t bf,
                                                   int64_t q_ppm, Div64 div_q) {
    unsigned ignored = 0;                                    // (the serve pass has already vetted every service time)
    return serve_terms(rs, mp, addr, issue, bf, q_ppm, div_q, ignored, 33);
}

struct FixRun { int64_t B, Bs; long long dstall, max_c; bool settled; };
__device__ __forceinline__ void fix_entry(FixRun &f, const InHead &h, int64_t *completion, int64_t *stall) {
    if (f.settled) return;
    if (f.B <= h.m - h.s) { f.settled = true; return; }      // idle on arrival: from here on the as-if run was right
    f.B += h.s;                                              // it waited for the queue: starts at B
    f.Bs = max(f.Bs + h.s, h.m);
    const bool op = (h.xo >> 31) != 0u;
    const int64_t xfer = (int64_t)(h.xo & 0x7fffffffu);
    const int64_t done = f.B + (op ? 0 : xfer);
    f.dstall += f.B - f.Bs;                                  // completion moved from Bs + post to B + post
    completion[h.idx] = done; stall[h.idx] = done - (h.m - h.s - (op ? xfer : 0));
    f.max_c = max(f.max_c, (long long)done);
}

constexpr int kInStrThreads = 512;
constexpr int kInStrWarps = kInStrThreads / 32;
constexpr int kInStrQItems = 32;                          // records per thread and turn inside the queue-number prefix
constexpr int kInStrQChunk = kInStrThreads * kInStrQItems;
constexpr int kInStrKeep = 1024;                          // kept records served at a time (a chunk with more is served in windows)
constexpr int kInStrMaxStragglers = 255;                   // a tile with as many is served again whole instead (a queue's place, plus one, is a byte)
constexpr int kInStrList = 32;                            // records of one queue in a window that its list holds (more: the window is scanned)
constexpr int kInStrQueuesPerThread = (kInMaxQueues + kInStrThreads - 1) / kInStrThreads;
static_assert(kInStrQChunk <= 65536, "a kept record's position in its chunk is stored in 16 bits");
static_assert(kInQidPrefix % kInStrQChunk == 0 && kInStrQItems == 32, "a thread's 32 queue numbers are four 16-byte loads");

template <bool DEBT>
__global__ void __launch_bounds__(kInStrThreads, 2)
k_inorder_fixstraggle(const hbf_access_t *__restrict__ acc, uint64_t n, const __grid_constant__ InTileMap tmap,
                      const RangeSnap *__restrict__ ranges_g, const __grid_constant__ ModelParams mp_arg,
                      const __grid_constant__ FastRange fast_arg, BatchCtrl *ctrl,
                      const int64_t *__restrict__ in_bin, const InHead *__restrict__ in_head,
                      const uint8_t *__restrict__ in_headcnt, int64_t *completion, int64_t *stall, InTile *in_tile,
                      const unsigned long long *claim_limit_p, const uint16_t *__restrict__ in_qid, uint32_t qid_stride,
                      const uint32_t head_depth, TileBalance *bal) {
    extern __shared__ __align__(16) unsigned char str_smem[];
    __shared__ ModelParams mp;
    __shared__ FastRange fast_range;
    __shared__ uint32_t s_cells[kInStrWarps];
    __shared__ uint32_t s_total;
    __shared__ uint32_t s_stragglers;                        // straggling queues of the tile
    __shared__ int s_open;                                   // those whose two runs have not met yet
    __shared__ long long s_red[2];

    if (ctrl->skip || ctrl->run_sort || !ctrl->inorder_used) return;
    const uint32_t tile = blockIdx.x;
    if (tile == 0u) return;                                  // the first tile was served from its true entering state
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const RangeSnap &rs = *ranges_g;
    const uint32_t R = mp_arg.n_queues;
    int64_t *Bt = reinterpret_cast<int64_t *>(str_smem);                       // [queues] true run
    int64_t *Ba = Bt + kInMaxQueues;                                           // [queues] as-if-idle run
    longlong2 *ent_as = reinterpret_cast<longlong2 *>(Ba + kInMaxQueues);      // [keep] kept records, batch order: issue time, service time
    uint2 *ent_pq = reinterpret_cast<uint2 *>(ent_as + kInStrKeep);            //        transfer | op << 31, queue | position << 16
    uint16_t *oq = reinterpret_cast<uint16_t *>(ent_pq + kInStrKeep);          // [stragglers] their queues
    uint8_t *open = reinterpret_cast<uint8_t *>(oq + kInMaxQueues);            // [2 x queues] 0, or 1 + the queue's place in oq while its runs have not met
    uint16_t *lst = reinterpret_cast<uint16_t *>(open + 2 * kInMaxQueues);     // [stragglers][kInStrList] the window's records of each queue
    uint32_t *lcount = reinterpret_cast<uint32_t *>(lst + kInStrMaxStragglers * kInStrList);   // [stragglers] how many
    __shared__ uint32_t s_overflow;
    if (tid < kInStrMaxStragglers) lcount[tid] = 0u;
    if (tid == 0) { mp = mp_arg; fast_range = fast_arg; s_stragglers = 0u; s_total = 0u; s_overflow = 0u; s_red[0] = 0; s_red[1] = INT64_MIN; }
    __syncthreads();

    // ---- fix-up, first entry: this thread's queues of the tile, their loads issued side by side.  Four queues in five
    // are idle when their first access of the tile arrives: they are done here.  The others go on a list.
    long long dstall = 0, max_c = INT64_MIN;
    uint16_t *deep = reinterpret_cast<uint16_t *>(ent_pq);   // [queues] the list (the record windows are not in use yet)
    {
        uint32_t c[kInStrQueuesPerThread]; int64_t Bin[kInStrQueuesPerThread];
        InHead e0[kInStrQueuesPerThread];
#pragma unroll
        for (int k = 0; k < kInStrQueuesPerThread; ++k) {
            const uint32_t q = (uint32_t)(k * kInStrThreads + tid);
            c[k] = 0u; Bin[k] = kNegInf;
            if (q < R) { c[k] = in_headcnt[(uint64_t)tile * R + q]; Bin[k] = in_bin[(uint64_t)tile * R + q]; }
        }
#pragma unroll
        for (int k = 0; k < kInStrQueuesPerThread; ++k)
            if (c[k] > 0u) e0[k] = in_head[head_slot(tile, R, (uint32_t)(k * kInStrThreads + tid), 0u)];
#pragma unroll
        for (int k = 0; k < kInStrQueuesPerThread; ++k) {
            const uint32_t q = (uint32_t)(k * kInStrThreads + tid);
            if (q < kInMaxQueues) { open[q] = 0; open[kInMaxQueues + q] = 0; Ba[q] = kNegInf; Bt[q] = Bin[k]; }   // (upper half: not modeled, or not defined)
            if (c[k] == 0u) continue;
            if (Bin[k] <= e0[k].m - e0[k].s) continue;       // idle on arrival: the as-if run was right from the start
            deep[atomicAdd(&s_total, 1u)] = (uint16_t)q;
        }
    }
    __syncthreads();
    // ---- fix-up, the rest: one thread per listed queue walks its head entries (fetched in two rounds) from the true
    // entering busy-until until an access arrives on an idle queue
    {
        const uint32_t n_deep = s_total;
        for (uint32_t d = (uint32_t)tid; d < n_deep; d += kInStrThreads) {
            const uint32_t q = deep[d];
            const uint64_t idx = (uint64_t)tile * R + q;
            const uint32_t c = in_headcnt[idx];
            const InHead *h = in_head + head_slot(tile, R, q, 1u) - 1;       // h[j], j >= 1: the queue's later entries, side by side
            FixRun f; f.B = Bt[q]; f.Bs = kNegInf; f.dstall = 0; f.max_c = INT64_MIN; f.settled = false;
            InHead g[4];
            g[0] = in_head[head_slot(tile, R, q, 0u)];       // (listed queues have at least one entry)
#pragma unroll
            for (int j = 1; j < 4; ++j) if ((uint32_t)j < c) g[j] = h[j];
#pragma unroll
            for (int j = 0; j < 4; ++j) if ((uint32_t)j < c) fix_entry(f, g[j], completion, stall);
            if (!f.settled && c > 4u) {
#pragma unroll
                for (int j = 4; j < kInHead; ++j) if ((uint32_t)j < c) g[j - 4] = h[j];
#pragma unroll
                for (int j = 4; j < kInHead; ++j) if ((uint32_t)j < c) fix_entry(f, g[j - 4], completion, stall);
            }
            max_c = max(max_c, f.max_c);                     // (true completions: valid whoever writes them last)
            if (!f.settled && c == head_depth) {
                // still backlogged after its head entries: the loop below serves this queue again from the tile's
                // start (Bt[q] still holds the entering value) and accounts for all of its corrections
                const uint32_t place = atomicAdd(&s_stragglers, 1u);
                oq[place] = (uint16_t)q;
                open[q] = (uint8_t)min(place + 1u, 255u);   // (a tile with more than kInStrMaxStragglers - 1 of them leaves below)
            } else {
                dstall += f.dstall;
            }
        }
    }
    __syncthreads();
    const uint32_t stragglers = s_stragglers;
    if (bal && tid == 0) {                                   // what the number of head entries of later batches follows from
        atomicMax(&bal->strag_max, stragglers);
        if (stragglers >= min(max(8u, R / 4u), (uint32_t)kInStrMaxStragglers)) atomicAdd(&bal->strag_flagged, 1u);
    }
    // many queues far behind: the re-serve pass takes the whole tile (one block serves it again from end to end, which costs
    // as much as the serve pass itself, so the bar is as high as this loop's tables allow)
    if (stragglers >= min(max(8u, R / 4u), (uint32_t)kInStrMaxStragglers)) {
        if (tid == 0) in_tile[tile].reserve = 1u;
        return;
    }
    if (stragglers > 0u) {
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const bool one_range = fast_arg.on != 0u && mp_arg.pow2_geom != 0u;
    const bool fast_terms = one_range && mp_arg.xfer_tab_max_cb != 0u && q_ppm == 1000000;
    const uint64_t claim_limit = DEBT ? *claim_limit_p : 0ull;     // as in the serve pass
    const int64_t quantum_ns = !DEBT ? 0 : q_ppm == 1000000 ? mp_arg.t_read_ns + mp_arg.t_prog_ns
        : (int64_t)div64((uint64_t)(mp_arg.t_read_ns + mp_arg.t_prog_ns) * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);
    const uint64_t tile_begin = tile_first(tmap, tile), tile_end = tile_last(tmap, tile);
    const uint32_t tile_len = (uint32_t)(tile_end - tile_begin);       // offsets inside a tile fit 32 bits
    const hbf_access_t *acc_t = acc + tile_begin;
    const uint4 *qid_t = reinterpret_cast<const uint4 *>(in_qid + (uint64_t)tile * qid_stride);
    if (tid == 0) s_open = (int)stragglers;

    // the queue numbers of the next chunk are on their way while this one is filtered
    // (only the queue numbers: past the prefix, a rare stretch, the addresses are loaded when they are needed)
    uint4 nx_q[kInStrQItems / 8];
    auto fetch = [&](uint32_t cb) {
        if (cb < tile_len && cb + kInStrQChunk <= qid_stride) {
#pragma unroll
            for (int k = 0; k < kInStrQItems / 8; ++k) nx_q[k] = __ldg(qid_t + (cb >> 3) + tid * (kInStrQItems / 8) + k);
        }
    };
    // the kept records of a window, one per thread (their positions in the chunk are in the window already): the records are
    // fetched side by side, their terms computed once, and they take their places in the window
    constexpr int kPerThread = kInStrKeep / kInStrThreads;
    auto fill_window = [&](uint32_t cb, uint32_t wn) {
        uint64_t r_addr[kPerThread], r_bf[kPerThread]; int64_t r_issue[kPerThread]; uint32_t r_e[kPerThread];
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const uint32_t slot = (uint32_t)(k * kInStrThreads + tid);
            if (slot < wn) {
                r_e[k] = ent_pq[slot].y;
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc_t + cb + r_e[k]);
                r_addr[k] = __ldg(rec); r_issue[k] = (int64_t)__ldg(rec + 1); r_bf[k] = __ldg(rec + 2);
            }
        }
#pragma unroll
        for (int k = 0; k < kPerThread; ++k) {
            const uint32_t slot = (uint32_t)(k * kInStrThreads + tid);
            if (slot < wn) {
                Served v = fast_terms ? serve_terms_fast(fast_range, mp, r_addr[k], r_issue[k], r_bf[k])
                                      : serve_terms_general(rs, mp, r_addr[k], r_issue[k], r_bf[k], q_ppm, div_q);
                if (DEBT && tile_begin + cb + r_e[k] < claim_limit) v.s += quantum_ns;
                ent_as[slot] = make_longlong2(r_issue[k], v.s);
                ent_pq[slot] = make_uint2(v.xfer | (v.op << 31), v.queue | (r_e[k] << 16));
                const uint32_t place = open[v.queue];         // (0: the queue's runs met in an earlier window of this chunk)
                if (place) {
                    const uint32_t at = atomicAdd(&lcount[place - 1u], 1u);
                    if (at < (uint32_t)kInStrList) lst[(place - 1u) * kInStrList + at] = (uint16_t)slot; else s_overflow = 1u;
                }
            }
        }
    };
    fetch(0u);

    uint32_t cb = 0;
    while (cb < tile_len) {
        const bool by_qid = cb + kInStrQChunk <= qid_stride;  // the same for the whole block
        // ---- keep the modeled records of the open queues, in batch order: bit j of `keep` is this thread's item j, the
        // thread's items being 32 consecutive records
        uint32_t keep = 0;
        if (by_qid) {
            // (numbers past the tile's end are not defined: the table is indexed by 12 bits, twice the queues, and whatever
            // such a number finds there is masked off by position)
#pragma unroll
            for (int j = 0; j < kInStrQItems; ++j) {
                const uint4 v = nx_q[j >> 3];
                const uint32_t w = ((j >> 1) & 3) == 0 ? v.x : ((j >> 1) & 3) == 1 ? v.y : ((j >> 1) & 3) == 2 ? v.z : v.w;
                keep |= open[(w >> (16 * (j & 1))) & (2u * kInMaxQueues - 1u)] != 0 ? 1u << j : 0u;
            }
            const uint32_t room = tile_len - cb, mine = (uint32_t)(tid * kInStrQItems);   // records of the tile from this chunk on
            const uint32_t have = room > mine ? min(room - mine, (uint32_t)kInStrQItems) : 0u;
            keep &= have >= 32u ? 0xffffffffu : (1u << have) - 1u;
            fetch(cb + kInStrQChunk);
        } else {
            // past the prefix (a rare stretch: its size matters more than its speed) the queue comes from the record
#pragma unroll 2
            for (int j = 0; j < kInStrQItems; ++j) {
                const uint32_t i = cb + (uint32_t)(tid * kInStrQItems + j);
                if (i < tile_len) {
                    const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc_t + i);
                    const uint64_t addr = __ldg(rec);
                    bool k;
                    if (one_range) {
                        const uint32_t q = fast_queue(fast_range, mp, addr);
                        k = q != 0xffffffffu && open[q] != 0;
                    } else {
                        const Served v = serve_terms_general(rs, mp, addr, (int64_t)__ldg(rec + 1), __ldg(rec + 2), q_ppm, div_q);
                        k = v.st == HBF_ST_READY && open[v.queue] != 0;
                    }
                    keep |= k ? 1u << j : 0u;
                }
            }
            fetch(cb + kInStrQChunk);
        }
        uint32_t first;                                      // place of this thread's first kept record among the chunk's
        {
            const uint32_t cnt = (uint32_t)__popc(keep);
            uint32_t incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
            if (lane == 31) s_cells[warp] = incl;
            __syncthreads();
            if (warp == 0) {
                const uint32_t c = lane < kInStrWarps ? s_cells[lane] : 0u;
                uint32_t in2 = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, in2, o); if (lane >= o) in2 += t; }
                if (lane < kInStrWarps) s_cells[lane] = in2 - c;
                if (lane == 31) s_total = in2;
            }
            __syncthreads();
            first = s_cells[warp] + incl - cnt;
        }
        // ---- the kept records, a window of kInStrKeep at a time (one window, nearly always)
        const uint32_t total = s_total;
        for (uint32_t wb = 0; wb < total; wb += (uint32_t)kInStrKeep) {
            const uint32_t wn = min(total - wb, (uint32_t)kInStrKeep);
            {
                uint32_t m = keep;
                while (m) {
                    const uint32_t j = (uint32_t)__ffs((int)m) - 1u;
                    m &= m - 1u;
                    const uint32_t slot = first + (uint32_t)__popc(keep & ((1u << j) - 1u)) - wb;   // (wraps below the window)
                    if (slot < wn) ent_pq[slot].y = (uint32_t)(tid * kInStrQItems) + j;
                }
            }
            __syncthreads();
            fill_window(cb, wn);
            __syncthreads();
            // Every straggling queue has the window's records of its own in a short list (in the order the threads happened
            // to append them): one thread per queue sorts its list by position (the window is in batch order) and re-serves
            // them, carrying the two runs.
            auto reserve_one = [&](uint32_t kk, int64_t &BT, int64_t &BA, bool writer) {
                const uint2 pq = ent_pq[kk];
                const longlong2 as = ent_as[kk];
                const int64_t xfer = (int64_t)(pq.x & 0x7fffffffu);
                const bool op = (pq.x >> 31) != 0u;
                const int64_t a = as.x + (op ? xfer : 0);
                BT = max(a, BT) + as.y; BA = max(a, BA) + as.y;
                if (BT != BA && writer) {                     // the serve pass wrote BA + post
                    const uint64_t i = min(tile_begin + cb + (pq.y >> 16), tile_end - 1);
                    const int64_t done = BT + (op ? 0 : xfer);
                    completion[i] = done; stall[i] = done - as.x;
                    dstall += BT - BA; max_c = max(max_c, (long long)done);
                }
            };
            if (!s_overflow) {
                for (uint32_t t = (uint32_t)tid; t < stragglers; t += kInStrThreads) {
                    const uint32_t q = oq[t];
                    const uint32_t cnt = lcount[t];
                    lcount[t] = 0u;
                    if (!open[q] || cnt == 0u) continue;
                    uint16_t *mine = lst + t * kInStrList;
                    for (uint32_t i = 1; i < cnt; ++i) {      // a handful of entries: insertion sort
                        const uint16_t key = mine[i];
                        uint32_t j = i;
                        while (j > 0u && mine[j - 1u] > key) { mine[j] = mine[j - 1u]; --j; }
                        mine[j] = key;
                    }
                    int64_t BT = Bt[q], BA = Ba[q];
                    for (uint32_t i = 0; i < cnt; ++i) reserve_one(mine[i], BT, BA, true);
                    Bt[q] = BT; Ba[q] = BA;
                    if (BT == BA) { open[q] = 0; atomicSub(&s_open, 1); }   // the runs have met: the rest of the tile was served right
                }
            } else {
                // some queue has more records in this window than a list holds: one warp per straggling queue scans the
                // window 32 records at a time and re-serves its own in order; every lane carries the two runs, lane 0 writes
                for (uint32_t t = (uint32_t)warp; t < stragglers; t += kInStrWarps) {
                    const uint32_t q = oq[t];
                    if (lane == 0) lcount[t] = 0u;
                    if (!open[q]) continue;
                    int64_t BT = Bt[q], BA = Ba[q];
                    for (uint32_t k0 = 0; k0 < wn; k0 += 32u) {
                        const uint32_t k = k0 + (uint32_t)lane;
                        unsigned hits = __ballot_sync(0xffffffffu, k < wn && (ent_pq[min(k, wn - 1u)].y & 0xffffu) == q);
                        while (hits) {
                            const uint32_t kk = k0 + (uint32_t)__ffs((int)hits) - 1u;
                            hits &= hits - 1u;
                            reserve_one(kk, BT, BA, lane == 0);
                        }
                    }
                    if (lane == 0) {
                        Bt[q] = BT; Ba[q] = BA;
                        if (BT == BA) { open[q] = 0; atomicSub(&s_open, 1); }
                    }
                }
                __syncthreads();
                if (tid == 0) s_overflow = 0u;
            }
            __syncthreads();
        }
        if (*reinterpret_cast<volatile int *>(&s_open) <= 0) break;
        cb += kInStrQChunk;
    }
    }
    dstall = warp_sum(dstall); max_c = warp_max(max_c);
    if (lane == 0) {
        if (dstall) atomicAdd((unsigned long long *)&s_red[0], (unsigned long long)dstall);
        if (max_c != INT64_MIN) atomicMax(&s_red[1], max_c);
    }
    __syncthreads();
    if (tid == 0) {
        if (s_red[0]) in_tile[tile].fix_delta = s_red[0];    // (cleared by the serve pass; this block is the tile's only writer)
        if (s_red[1] != INT64_MIN) atomicMax(&ctrl->max_completion_ns, s_red[1]);
    }
}

#ifndef HBF_IN_SKEW_PERMILLE
#define HBF_IN_SKEW_PERMILLE 60
#endif
// One wave of resident blocks: as many tiles as the device holds serve blocks.  When the batch is large enough to fill
// that wave, the tiles of the blocks that the hardware favours (one per SM) are larger by the skew, the others smaller,
// so that both blocks of an SM finish together.
InTileMap inorder_tile_map(uint64_t n, int sm_count, bool by_table) {
    InTileMap m{};
    m.n = n;
    const uint64_t sms = (uint64_t)std::max(1, sm_count);
    const uint64_t want_tiles = std::min<uint64_t>(kInMaxTiles, sms * kInBlocksPerSM);
    auto round_up = [](uint64_t v) { return std::max<uint64_t>((v + kInTileQuantum - 1) / kInTileQuantum * kInTileQuantum, kInTileQuantum); };
    const uint64_t even = round_up((n + want_tiles - 1) / want_tiles);
    if (kInBlocksPerSM == 2 && want_tiles == 2 * sms && even >= 64 * kInTileQuantum && HBF_IN_SKEW_PERMILLE > 0) {
        const uint64_t big = round_up(even * (1000 + HBF_IN_SKEW_PERMILLE) / 1000);
        if (by_table && 2 * sms <= kInBalMax) {
            // exactly two tiles per SM, their places in a table (launch_inorder writes it: the two nominal sizes until
            // measurements are at hand); big and small are the nominal sizes only
            m.n_big = (uint32_t)sms; m.n_tiles = (uint32_t)(2 * sms); m.big = (uint32_t)big;
            m.small = (uint32_t)round_up(even * (1000 - HBF_IN_SKEW_PERMILLE) / 1000);
            m.max_tile = (uint32_t)round_up(even * 1200 / 1000); m.by_sm = 1u;
            return m;
        }
        if (big * sms < n) {
            const uint64_t rest = n - big * sms;
            const uint64_t small = round_up((rest + sms - 1) / sms);
            m.n_big = (uint32_t)sms; m.big = (uint32_t)big; m.small = (uint32_t)small;
            m.n_tiles = (uint32_t)(sms + (rest + small - 1) / small);
            m.max_tile = (uint32_t)std::max(big, small);
            return m;
        }
    }
    m.n_big = 0; m.big = m.small = (uint32_t)even;
    m.n_tiles = (uint32_t)((n + even - 1) / even);
    m.max_tile = (uint32_t)even;
    return m;
}

// Where n_tiles tiles begin when tile t gets the share share[t] of a batch of n records, in whole quanta (every tile at
// least one); first[n_tiles] >= n.
static void tiles_from_shares(const double *share, uint32_t n_tiles, uint64_t n, uint32_t *first, uint32_t *max_tile) {
    double sum_share = 0.0;
    for (uint32_t t = 0; t < n_tiles; ++t) sum_share += share[t];
    const uint64_t quanta = (n + kInTileQuantum - 1) / kInTileQuantum;
    uint64_t q[kInBalMax], used = 0;
    for (uint32_t t = 0; t < n_tiles; ++t) { q[t] = std::max<uint64_t>(1, (uint64_t)(share[t] / sum_share * (double)quanta)); used += q[t]; }
    for (uint32_t t = 0; used < quanta; t = (t + 1) % n_tiles) { ++q[t]; ++used; }           // what rounding down left over
    for (uint32_t t = 0; used > quanta; t = (t + 1) % n_tiles) if (q[t] > 1) { --q[t]; --used; }
    uint64_t at = 0, largest = 0;
    for (uint32_t t = 0; t < n_tiles; ++t) { first[t] = (uint32_t)(at * kInTileQuantum); at += q[t]; largest = std::max(largest, q[t]); }
    first[n_tiles] = (uint32_t)(at * kInTileQuantum);
    *max_tile = (uint32_t)(largest * kInTileQuantum);
}

// Shares from the record an earlier batch left (see TileBalance): every tile in proportion to the rate measured at its
// place, blended with the share it had (so that one odd measurement moves a tile by little), within 15 % of the mean.
// False when the record is not a complete measurement of one batch with this many tiles.
static bool measured_shares(const TileBalance &rec, uint32_t n_tiles, double *share) {
    double rate[kInBalMax], sum_rate = 0.0, sum_len = 0.0;
    for (uint32_t t = 0; t < n_tiles; ++t) {
        if (rec.claim[t] != rec.claim[0] || rec.claim[t] == 0u || rec.ns[t] == 0u || rec.len[t] == 0u) return false;
        rate[t] = (double)rec.len[t] / (double)rec.ns[t];
        sum_rate += rate[t]; sum_len += (double)rec.len[t];
    }
    const double mean = 1.0 / n_tiles;
    for (uint32_t t = 0; t < n_tiles; ++t) {
        const double s = 0.3 * ((double)rec.len[t] / sum_len) + 0.7 * (rate[t] / sum_rate);
        share[t] = std::min(std::max(s, 0.85 * mean), 1.15 * mean);
    }
    return true;
}

// dynamic shared memory of the serve kernel: the per-queue state, the per-die counters, every warp's tables of lane numbers
size_t inorder_serve_smem(uint32_t n_dies) { return (size_t)kInMaxQueues * 16 + (size_t)n_dies * 28 + (size_t)kInWarps * kInRows * kInTagStride; }
static size_t inorder_straggle_smem() {
    return (size_t)kInMaxQueues * 16 + (size_t)kInStrKeep * 24 + (size_t)kInMaxQueues * 4 + (size_t)kInStrMaxStragglers * (kInStrList * 2 + 4);
}

// ======================================================================================================
// Small batches (at most kInSmallMax records, in issue order) are served exactly in one launch, instead of tiles, a scan, a
// fix-up and a straggle pass whose fixed costs a few thousand records cannot pay for.  Queues do not interact, so the
// queues are dealt to the blocks in slices of 64 consecutive ones, and a block serves its slice on its own; no block
// waits for another.  Every block reads ALL the records (a few hundred KB, from the L2 after the first block):
//   terms   every thread takes records i, i + 1024, ...: status, queue, service terms (the short form for the common
//           configuration, else the general one).  Every block counts the statuses of the whole batch, so all blocks
//           take the same decision about it; a record of the block's slice leaves service and transfer in shared
//           memory by batch index and gets the sort key (queue in the slice) << 14 | index << 1 | op; the others all ones
//   sort    one stable radix pass over the 6 queue bits of the slice, in shared memory: a warp owns consecutive keys and
//           ranks them 32 at a time (match_any); keys of other slices go behind every queue
//   serve   a segmented max-plus scan over the slice's sorted keys (a queue's run is a segment): every thread owns up to 8
//           consecutive entries, composes their maps, the block scans the threads' maps, and the thread walks its
//           entries again from the busy-until that reaches it; per-die totals are summed along the runs (a die's
//           queues are neighbours)
// Statuses and the results of records that are not modeled are written by the block whose turn the record's round is.
// A batch that is not in issue order is handed to the sort path exactly as the tiled path hands it over.
// ======================================================================================================
constexpr int kInSmallThreads = 1024;
constexpr int kInSmallWarps = kInSmallThreads / 32;
constexpr uint32_t kInSmallItems = kInSmallMax / kInSmallThreads;          // sorted entries per thread, at most
constexpr uint32_t kInSmallIdxBits = 13, kInSmallQShift = kInSmallIdxBits + 1;
constexpr uint32_t kInSmallSlice = 64;                                     // queues per block: the bins of the radix pass, plus one for the rest
static_assert((1u << kInSmallIdxBits) == kInSmallMax, "index << 1 | op fits below the queue bits of the key");
static_assert(kInSmallMax % (kInSmallWarps * 32) == 0 && kInSmallWarps == 32, "a warp sorts whole rounds of 32 keys; a lane per warp in the offsets' scan");

size_t inorder_small_smem() { return (size_t)kInSmallMax * (8 + 4 + 4 + 4); }
uint32_t inorder_small_blocks(uint32_t n_queues) { return (n_queues + kInSmallSlice - 1) / kInSmallSlice; }

// one stable pass: src -> dst by the queue bits of the key; keys that are all ones take the extra bin behind every queue
__device__ __forceinline__ void small_radix_pass(const uint32_t *src, uint32_t *dst, uint32_t padded,
                                                 uint32_t (*hist)[kInSmallSlice + 1], uint32_t *dbase) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t per_warp = padded / kInSmallWarps;                      // (padded is a multiple of 1024)
    auto digit = [&](uint32_t key) { return key == 0xffffffffu ? kInSmallSlice : key >> kInSmallQShift; };
    for (uint32_t e = tid; e < kInSmallWarps * (kInSmallSlice + 1); e += kInSmallThreads) (&hist[0][0])[e] = 0u;
    __syncthreads();
    for (uint32_t r = 0; r < per_warp; r += 32u) {                         // counts per (warp, digit)
        const uint32_t d = digit(src[warp * per_warp + r + lane]);
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        if (lane == __ffs(peers) - 1) hist[warp][d] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    // where the keys of (digit, warp) begin: digits in order, within a digit the warps in order
    for (uint32_t d = warp; d <= kInSmallSlice; d += kInSmallWarps) {      // lane = the warp whose count this is
        const uint32_t v = hist[lane][d];
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        hist[lane][d] = inc - v;
        if (lane == 31) dbase[d] = inc;
    }
    __syncthreads();
    if (warp == 0) {                                                       // exclusive scan of the 65 digit totals: three per lane
        uint32_t v[3], sum = 0;
#pragma unroll
        for (int k = 0; k < 3; ++k) { const uint32_t d = lane * 3 + k; v[k] = d <= kInSmallSlice ? dbase[d] : 0u; sum += v[k]; }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += t; }
        uint32_t run = inc - sum;
#pragma unroll
        for (int k = 0; k < 3; ++k) { const uint32_t d = lane * 3 + k; if (d <= kInSmallSlice) dbase[d] = run; run += v[k]; }
    }
    __syncthreads();
    for (uint32_t r = 0; r < per_warp; r += 32u) {                         // scatter, 32 keys at a time, in order
        const uint32_t key = src[warp * per_warp + r + lane], d = digit(key);
        const unsigned peers = __match_any_sync(0xffffffffu, d);
        const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
        dst[dbase[d] + hist[warp][d] + rank] = key;
        __syncwarp();
        if (lane == __ffs(peers) - 1) hist[warp][d] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
}

template <bool DEBT>
__global__ void __launch_bounds__(kInSmallThreads, 1)
k_small_serve(const hbf_access_t *__restrict__ acc, const uint32_t n, const RangeSnap *__restrict__ ranges_g,
              const ModelParams *__restrict__ mp_g, const __grid_constant__ FastRange fast_arg, BatchCtrl *ctrl,
              uint8_t *__restrict__ status, int64_t *__restrict__ completion,
              int64_t *__restrict__ stall, hbf_die_stats_t *stats_stage, const int64_t *__restrict__ busy, int64_t *busy_stage,
              InTile *in_tile, const unsigned long long *claim_limit_p, uint32_t *die_claims, int forced) {
    extern __shared__ __align__(16) unsigned char sm_small[];
    __shared__ RangeSnap rs;
    __shared__ ModelParams mp;
    __shared__ FastRange fast_range;
    __shared__ unsigned long long s_cnt[4];                  // of the whole batch: native, ready, failing; ready in this block's slice
    __shared__ uint32_t s_unsorted;
    __shared__ long long s_tot[3];                           // of the slice: stalls, services, largest completion
    __shared__ uint32_t s_hist[kInSmallWarps][kInSmallSlice + 1];
    __shared__ uint32_t s_dbase[kInSmallSlice + 1];
    __shared__ int64_t w_S[kInSmallWarps], w_M[kInSmallWarps];
    __shared__ int w_f[kInSmallWarps];
    // (a flag another block of this launch may just have set takes the same decision this block is about to take)
    if (ctrl->skip || ctrl->run_sort) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t slice = blockIdx.x, n_slices = gridDim.x, q_lo = slice * kInSmallSlice;
    int64_t *s_s = reinterpret_cast<int64_t *>(sm_small);                     // [kInSmallMax] service time, by batch index
    uint32_t *s_px = reinterpret_cast<uint32_t *>(s_s + kInSmallMax);        //               transfer | op << 31
    uint32_t *s_key = s_px + kInSmallMax, *s_key2 = s_key + kInSmallMax;      //               the keys and the sort's second buffer
    for (int i = tid; i < (int)(sizeof(RangeSnap) / 4); i += kInSmallThreads)
        reinterpret_cast<uint32_t *>(&rs)[i] = reinterpret_cast<const uint32_t *>(ranges_g)[i];
    for (int i = tid; i < (int)(sizeof(ModelParams) / 4); i += kInSmallThreads)
        reinterpret_cast<uint32_t *>(&mp)[i] = reinterpret_cast<const uint32_t *>(mp_g)[i];
    if (tid < 4) s_cnt[tid] = 0;
    if (tid < 3) s_tot[tid] = tid == 2 ? INT64_MIN : 0;
    if (tid == 0) { s_unsorted = 0u; fast_range = fast_arg; }
    const uint32_t padded = (n + kInSmallThreads - 1u) / kInSmallThreads * kInSmallThreads;     // whole rounds for every warp
    __syncthreads();

    // ---- terms
    const int64_t q_ppm = ctrl->q_ppm;
    const Div64 div_q = ctrl->div_q;
    const bool fast_terms = fast_arg.on != 0u && mp.pow2_geom != 0u && mp.xfer_tab_max_cb != 0u && q_ppm == 1000000;
    const uint64_t claim_limit = DEBT ? *claim_limit_p : 0ull;
    const int64_t quantum_ns = !DEBT ? 0 : q_ppm == 1000000 ? mp.t_read_ns + mp.t_prog_ns
        : (int64_t)div64((uint64_t)(mp.t_read_ns + mp.t_prog_ns) * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);
    uint32_t c_native = 0, c_ready = 0, c_fault = 0, c_unsorted = 0, c_mine = 0;
    long long sum_s = 0;
    for (uint32_t i0 = (uint32_t)tid; i0 < padded; i0 += 4u * kInSmallThreads) {
        uint64_t r_addr[4], r_bf[4]; int64_t r_issue[4], r_prev[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {                        // four records' loads go out together
            const uint32_t i = i0 + (uint32_t)k * kInSmallThreads;
            if (i < n) {
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + i);
                r_addr[k] = __ldg(rec); r_issue[k] = (int64_t)__ldg(rec + 1); r_bf[k] = __ldg(rec + 2);
                r_prev[k] = i > 0u ? (int64_t)__ldg(rec - 2) : INT64_MIN;
            }
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t i = i0 + (uint32_t)k * kInSmallThreads;
            if (i >= padded) break;
            uint32_t key = 0xffffffffu;                      // not modeled, another block's, or padding: behind every queue
            if (i < n) {
                const bool writer = (i / kInSmallThreads) % n_slices == slice;       // the block that writes what is not queue work
                if (r_issue[k] < r_prev[k]) c_unsorted = 1u;
                const Served v = fast_terms ? serve_terms_fast(fast_range, mp, r_addr[k], r_issue[k], r_bf[k])
                                            : serve_terms_general(rs, mp, r_addr[k], r_issue[k], r_bf[k], q_ppm, div_q);
                if (status && writer) status[i] = (uint8_t)v.st;
                if (v.st == HBF_ST_READY) {
                    ++c_ready;
                    if (v.queue - q_lo < kInSmallSlice) {    // (unsigned: queues below the slice wrap around)
                        ++c_mine;
                        int64_t sv = v.s;
                        if (DEBT && (uint64_t)i < claim_limit) sv += quantum_ns;
                        s_s[i] = sv; s_px[i] = v.xfer | (v.op << 31);
                        key = ((v.queue - q_lo) << kInSmallQShift) | (i << 1) | v.op;
                        sum_s += sv;
                    }
                } else if (v.st == HBF_ST_NATIVE) {
                    ++c_native;
                    if (writer) { completion[i] = r_issue[k]; stall[i] = 0; }
                } else {
                    ++c_fault;
                }
            }
            s_key[i] = key;
        }
    }
    c_native = (uint32_t)warp_sum((long long)c_native); c_ready = (uint32_t)warp_sum((long long)c_ready);
    c_fault = (uint32_t)warp_sum((long long)c_fault); c_mine = (uint32_t)warp_sum((long long)c_mine); sum_s = warp_sum(sum_s);
    c_unsorted = __any_sync(0xffffffffu, c_unsorted);
    if (lane == 0) {
        if (c_native) atomicAdd(&s_cnt[0], (unsigned long long)c_native);
        if (c_ready) atomicAdd(&s_cnt[1], (unsigned long long)c_ready);
        if (c_fault) atomicAdd(&s_cnt[2], (unsigned long long)c_fault);
        if (c_mine) atomicAdd(&s_cnt[3], (unsigned long long)c_mine);
        if (c_unsorted) atomicOr(&s_unsorted, 1u);
        if (sum_s) atomicAdd((unsigned long long *)&s_tot[1], (unsigned long long)sum_s);
    }
    __syncthreads();
    // what happens to the batch: the same decisions, in the same order, as the tiled path takes after its serve pass;
    // every block has seen every record and decides alike, the first one records it
    const bool fault = s_cnt[2] != 0ull, unsorted = s_unsorted != 0u;
    if (tid == 0 && slice == 0u) {
        ctrl->n_native = s_cnt[0]; ctrl->n_ready = s_cnt[1]; ctrl->n_fault = s_cnt[2];
        if (unsorted) ctrl->unsorted = 1u;
        if (fault) { ctrl->code = HBF_E_ACCESS_FAULT; ctrl->skip = 1; }                 // fail closed: refuse the batch
        else if (unsorted && forced) { ctrl->code = HBF_E_INVAL; ctrl->skip = 1; }
        else if (unsorted) ctrl->run_sort = 1u;                                         // hand the batch to the sort path
        else ctrl->inorder_used = 1u;
    }
    if (fault || unsorted) return;                           // nothing of the batch's state has been written yet

    // ---- sort the slice's keys by queue, stable (so a queue's records stay in batch order)
    small_radix_pass(s_key, s_key2, padded, s_hist, s_dbase);
    const uint32_t *sorted = s_key2;

    // ---- serve: a segmented max-plus scan over the sorted entries.  An entry is the map B -> max(B + s, a + s); the head
    // of a run starts from the busy-until earlier batches left on its queue, so its map no longer depends on what
    // comes in (f).
    const uint32_t m = (uint32_t)s_cnt[3];
    long long sum_stall = 0, max_c = INT64_MIN;
    {
        struct SMap { int64_t S, M; int f; };
        auto then = [](const SMap &x, const SMap &y) {         // x first, then y
            if (y.f) return y;
            SMap r; r.S = x.S + y.S; r.M = max((int64_t)(x.M + y.S), y.M); r.f = x.f; return r;
        };
        const uint32_t per = (m + kInSmallThreads - 1u) / kInSmallThreads;   // entries per thread (at most kInSmallItems)
        const uint32_t p0 = (uint32_t)tid * per;
        uint32_t key[kInSmallItems]; int64_t a[kInSmallItems], sv[kInSmallItems]; uint32_t px[kInSmallItems];
        int64_t issue[kInSmallItems]; uint32_t bytes[kInSmallItems];
        const uint32_t prev_q = p0 > 0u && p0 <= m ? sorted[p0 - 1u] >> kInSmallQShift : 0xffffffffu;
#pragma unroll
        for (uint32_t j = 0; j < kInSmallItems; ++j) {       // the issue times and sizes come from the records again, side by side
            const uint32_t p = p0 + j;
            key[j] = j < per && p < m ? sorted[p] : 0xffffffffu;
            if (key[j] != 0xffffffffu) {
                const uint64_t *rec = reinterpret_cast<const uint64_t *>(acc + ((key[j] >> 1) & (kInSmallMax - 1u)));
                issue[j] = (int64_t)__ldg(rec + 1); bytes[j] = (uint32_t)__ldg(rec + 2);
            }
        }
        // per-die totals along the thread's entries: a die's queues are neighbours in the sorted order
        uint32_t run_die = 0xffffffffu, run_n = 0, run_np = 0, run_cl = 0;
        unsigned long long run_busy = 0, run_br = 0, run_bp = 0;
        auto flush = [&]() {
            if (run_die == 0xffffffffu) return;
            // (the staging copy was cleared by the begin kernel; a handful of adds per thread; the energy follows from the
            // counts when the batch is committed)
            unsigned long long *g = reinterpret_cast<unsigned long long *>(stats_stage + run_die);
            atomicAdd(&g[0], run_busy);
            if (run_br) atomicAdd(&g[1], run_br);
            if (run_bp) atomicAdd(&g[2], run_bp);
            if (run_n - run_np) atomicAdd(&g[4], (unsigned long long)(run_n - run_np));
            if (run_np) atomicAdd(&g[5], (unsigned long long)run_np);
            if (DEBT && run_cl) atomicAdd(&die_claims[run_die], run_cl);
            run_busy = 0; run_br = 0; run_bp = 0; run_n = 0; run_np = 0; run_cl = 0;
        };
        SMap agg; agg.S = 0; agg.M = kNegInf; agg.f = 0;
#pragma unroll
        for (uint32_t j = 0; j < kInSmallItems; ++j) {
            if (key[j] != 0xffffffffu) {
                const uint32_t i = (key[j] >> 1) & (kInSmallMax - 1u), q = q_lo + (key[j] >> kInSmallQShift), op = key[j] & 1u;
                sv[j] = s_s[i]; px[j] = s_px[i];
                a[j] = issue[j] + (op ? (int64_t)(px[j] & 0x7fffffffu) : 0);
                const uint32_t before = j == 0u ? prev_q : key[j - 1u] >> kInSmallQShift;
                SMap e; e.S = sv[j]; e.f = before != (key[j] >> kInSmallQShift);
                e.M = (e.f ? max(a[j], busy[q]) : a[j]) + sv[j];
                agg = then(agg, e);
                const uint32_t die = mp.queue_level == 0u ? q / mp.planes : q;
                if (die != run_die) { flush(); run_die = die; }
                const uint32_t gs = op ? mp.prog_gran_shift : mp.read_gran_shift;
                const unsigned long long cb = (((unsigned long long)bytes[j] + (1ull << gs) - 1ull) >> gs) << gs;
                run_busy += (unsigned long long)sv[j]; ++run_n;
                if (op) { run_bp += cb; ++run_np; } else run_br += cb;
                if (DEBT && (uint64_t)i < claim_limit) ++run_cl;
            }
        }
        flush();
        // inclusive scan of the threads' maps across the warp, then across the warps
        SMap inc = agg;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            SMap u; u.S = __shfl_up_sync(0xffffffffu, inc.S, o); u.M = __shfl_up_sync(0xffffffffu, inc.M, o); u.f = __shfl_up_sync(0xffffffffu, inc.f, o);
            if (lane >= o) inc = then(u, inc);
        }
        if (lane == 31) { w_S[warp] = inc.S; w_M[warp] = inc.M; w_f[warp] = inc.f; }
        __syncthreads();
        SMap ex; ex.S = 0; ex.M = kNegInf; ex.f = 0;          // everything before this thread's entries
        for (int w = 0; w < warp; ++w) { SMap u; u.S = w_S[w]; u.M = w_M[w]; u.f = w_f[w]; ex = then(ex, u); }
        {
            SMap u; u.S = __shfl_up_sync(0xffffffffu, inc.S, 1); u.M = __shfl_up_sync(0xffffffffu, inc.M, 1); u.f = __shfl_up_sync(0xffffffffu, inc.f, 1);
            if (lane > 0) ex = then(ex, u);
        }
        // (the first entry of the slice is a head, so a map without a head never reaches an entry that needs its input)
        int64_t B = ex.M;
#pragma unroll
        for (uint32_t j = 0; j < kInSmallItems; ++j) {
            if (key[j] != 0xffffffffu) {
                const uint32_t i = (key[j] >> 1) & (kInSmallMax - 1u), lq = key[j] >> kInSmallQShift, op = key[j] & 1u;
                const uint32_t before = j == 0u ? prev_q : key[j - 1u] >> kInSmallQShift;
                if (before != lq) B = busy[q_lo + lq];
                B = max(a[j], B) + sv[j];
                const int64_t c = B + (op ? 0 : (int64_t)(px[j] & 0x7fffffffu)), waited = c - issue[j];
                completion[i] = c; stall[i] = waited;
                sum_stall += waited; max_c = max(max_c, (long long)c);
                const uint32_t p = p0 + j;
                const uint32_t after = p + 1u < m ? (j + 1u < per ? key[j + 1u] : sorted[p + 1u]) >> kInSmallQShift : 0xffffffffu;
                if (after != lq) busy_stage[q_lo + lq] = B;  // last access of its queue in this batch (the other queues keep the begin kernel's copy)
            }
        }
    }
    sum_stall = warp_sum(sum_stall); max_c = warp_max(max_c);
    if (lane == 0) { if (sum_stall) atomicAdd((unsigned long long *)&s_tot[0], (unsigned long long)sum_stall); atomicMax(&s_tot[2], max_c); }
    __syncthreads();
    if (tid == 0) {                                          // the slice's totals: one "tile" of the stall sum; the rest straight into the batch's
        InTile t; t.spec_sum = s_tot[0]; t.fix_delta = 0; t.true_sum = 0; t.reserve = 0u; t.stragglers = 0u; in_tile[slice] = t;
        if (s_tot[1]) atomicAdd((unsigned long long *)&ctrl->service_ns, (unsigned long long)s_tot[1]);
        if (s_tot[2] != INT64_MIN) atomicMax(&ctrl->max_completion_ns, s_tot[2]);
    }
}

bool inorder_small_batch(uint64_t n) { return n <= kInSmallMax; }

size_t inorder_head_bytes(uint64_t tiles, uint32_t n_queues) { return tiles * n_queues * (size_t)kInHead * sizeof(InHead); }

cudaError_t launch_inorder(const SubmitArgs &a, cudaStream_t st) {
    const uint64_t n = a.n;
    if (inorder_small_batch(n)) {                            // one launch, a block per 64 queues
        const bool debt = a.claim_limit != nullptr;
        const size_t smem = inorder_small_smem();
        cudaError_t e = ensure_dyn_smem((const void *)k_small_serve<false>, smem);
        if (e == cudaSuccess) e = ensure_dyn_smem((const void *)k_small_serve<true>, smem);
        if (e != cudaSuccess) return e;
        (debt ? k_small_serve<true> : k_small_serve<false>)<<<inorder_small_blocks(a.mp.n_queues), kInSmallThreads, smem, st>>>(
            a.acc, (uint32_t)n, a.ranges, a.mp_dev, a.fast, a.ctrl, a.status, a.completion, a.stall, a.stats_stage, a.busy, a.busy_stage,
            reinterpret_cast<InTile *>(a.ws.in_tile), a.claim_limit, a.die_claims, a.path == HBF_PATH_INORDER ? 1 : 0);
        g_kernel_launches += 1;
        return cudaGetLastError();
    }
    const bool by_table = a.bal && a.bal->on && a.bal->dev;
    InTileMap tmap = inorder_tile_map(n, a.sm_count, by_table);
    const unsigned n_tiles = tmap.n_tiles;
    // one full wave of two tiles per SM: the blocks take their tiles by SM and kind and leave their times; the tiles' places
    // come from a table in device memory: sized by the record of an earlier batch when there is a complete one, else in the
    // two nominal sizes
    TileBalanceHost *bal = tmap.by_sm ? a.bal : nullptr;
    uint32_t bal_seq = 0;
    if (bal) {
        bal_seq = ++bal->seq;
        if (bal_seq == 0u) bal_seq = ++bal->seq;             // (0 marks a tile never taken)
        double share[kInBalMax];
        if (!measured_shares(*bal->pinned, n_tiles, share))
            for (uint32_t t = 0; t < n_tiles; ++t) share[t] = t < tmap.n_big ? (double)tmap.big : (double)tmap.small;
        uint32_t first[kInBalMax + 1], max_tile = 0;
        tiles_from_shares(share, n_tiles, n, first, &max_tile);
        // (from pageable memory: the copy is staged before the call returns, so the array may go out of scope)
        cudaError_t e = cudaMemcpyAsync(bal->dev->first, first, (n_tiles + 1) * sizeof(uint32_t), cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return e;
        tmap.first = bal->dev->first; tmap.max_tile = max_tile;
    }
    // Head entries per (tile, queue).  Fewer cost the serve pass less (a shorter stretch of every tile with the head
    // bookkeeping, a smaller table) and leave more queues to the straggle pass; past 254 of those in a tile the tile is
    // served a second time.  So the number follows what the last batch needed: one fewer while no tile had 148 straggling
    // queues (an entry fewer leaves about 1.3 times as many: 100, 130, 164, 224 per tile with 6, 5, 4, 3 entries on the
    // capacity stream at half load, so 148 become about 200), one more above 200, all of them after a tile was served twice.  Results do not
    // depend on it.
    uint32_t depth = (uint32_t)kInHead;
    if (bal) {
        if (bal->depth == 0u || bal->depth > (uint32_t)kInHead) bal->depth = (uint32_t)kInHead;
        const TileBalance &rec = *bal->pinned;
        if (rec.strag_seq != 0u && rec.strag_seq != bal->depth_seen && rec.strag_depth == bal->depth) {
            bal->depth_seen = rec.strag_seq;
            if (rec.strag_flagged != 0u) bal->depth = (uint32_t)kInHead;
            else if (rec.strag_max > 200u && bal->depth < (uint32_t)kInHead) ++bal->depth;
            else if (rec.strag_max < 148u && bal->depth > 3u) --bal->depth;
        }
        depth = bal->depth_fixed != 0u ? std::min<uint32_t>(bal->depth_fixed, (uint32_t)kInHead) : bal->depth;
    } else if (a.bal && a.bal->depth_fixed != 0u) {
        depth = std::min<uint32_t>(a.bal->depth_fixed, (uint32_t)kInHead);
    }
    const uint64_t tile_records = tmap.max_tile;
    if (n_tiles > inorder_tiles_bound(n)) return cudaErrorInvalidValue;       // the workspace is carved for that many
    const uint32_t R = a.mp.n_queues, nd = a.mp.n_dies;
    const size_t smem_serve = inorder_serve_smem(nd), smem_str = inorder_straggle_smem();
    {
        const void *serve_fns[4] = {(const void *)k_inorder_serve<false, false>, (const void *)k_inorder_serve<true, false>,
                                    (const void *)k_inorder_serve<false, true>, (const void *)k_inorder_serve<true, true>};
        for (const void *f : serve_fns) { cudaError_t e = ensure_dyn_smem(f, smem_serve); if (e != cudaSuccess) return e; }
        cudaError_t e = ensure_dyn_smem((const void *)k_inorder_scan, 0);
        if (e != cudaSuccess) return e;
        e = ensure_dyn_smem((const void *)k_inorder_fixstraggle<false>, smem_str);
        if (e != cudaSuccess) return e;
        e = ensure_dyn_smem((const void *)k_inorder_fixstraggle<true>, smem_str);
        if (e != cudaSuccess) return e;
    }
    InTile *tiles = reinterpret_cast<InTile *>(a.ws.in_tile);
    InHead *heads = reinterpret_cast<InHead *>(a.ws.in_head);
    const bool debt = a.claim_limit != nullptr;              // retention on: the kernels that apply the claims
    const uint32_t qid_stride = (uint32_t)std::min<uint64_t>(tile_records, kInQidPrefix);
    if ((uint64_t)n_tiles * qid_stride > inorder_qid_entries(n)) return cudaErrorInvalidValue;
    auto serve = [&](bool reserve) {
        auto k = reserve ? (debt ? k_inorder_serve<true, true> : k_inorder_serve<true, false>)
                         : (debt ? k_inorder_serve<false, true> : k_inorder_serve<false, false>);
        k<<<n_tiles, kInThreads, smem_serve, st>>>(a.acc, n, tmap, a.ranges, a.mp, a.fast, a.ctrl, a.status, a.ws.in_agg,
                                                   a.stats_stage, a.completion, a.stall, a.ws.in_bin, tiles, heads, a.ws.in_headcnt,
                                                   a.busy, a.claim_limit, a.die_claims, debt ? *a.ret : RetDev{}, a.ws.in_qid, qid_stride,
                                                   bal ? bal->dev : nullptr, bal_seq, make_fast_geom(a.fast, a.mp), depth);
    };
    serve(false);
    k_inorder_scan<<<(R + kInScanQueues - 1) / kInScanQueues, dim3(kInScanQueues, kInScanChunks), 0, st>>>(
        a.ctrl, a.mp_dev, n_tiles, a.ws.in_agg, a.ws.in_bin, a.busy, a.busy_stage, a.stats_stage, a.path == HBF_PATH_INORDER ? 1 : 0);
    (debt ? k_inorder_fixstraggle<true> : k_inorder_fixstraggle<false>)<<<n_tiles, kInStrThreads, smem_str, st>>>(
        a.acc, n, tmap, a.ranges, a.mp, a.fast, a.ctrl, a.ws.in_bin, heads, a.ws.in_headcnt, a.completion, a.stall, tiles,
        a.claim_limit, a.ws.in_qid, qid_stride, depth, bal ? bal->dev : nullptr);
    serve(true);
    if (bal) {                                               // the tiles' times and straggler counts, for later batches; nothing waits for this copy
        cudaError_t e = cudaMemcpyAsync(bal->pinned, bal->dev, offsetof(TileBalance, first), cudaMemcpyDeviceToHost, st);
        if (e != cudaSuccess) return e;
    }
    g_kernel_launches += 4;
    return cudaGetLastError();
}

}  // namespace hbf
