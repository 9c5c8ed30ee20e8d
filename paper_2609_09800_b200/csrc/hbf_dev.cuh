// Internal declarations shared by the translation units of libhbf.so: device-side parameter blocks,
// the per-batch control block, and the host launchers of each kernel group.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/hbf.h"

namespace hbf {

constexpr int kMaxPasses = 8;            // 63 key bits / 8-bit digits
constexpr int kRadix = 256;
constexpr int kIssueBits = 47;           // key = queue << 47 | issue_ns
constexpr uint64_t kIssueMask = (1ull << kIssueBits) - 1;
constexpr int64_t kNegInf = INT64_MIN / 4;
constexpr uint32_t kSpinLimit = 1u << 24;  // polls of one look-back slot before giving up

// Sorted snapshot of the registered ranges (Design D1).
struct RangeSnap {
    uint64_t base[HBF_MAX_RANGES];
    uint64_t length[HBF_MAX_RANGES];
    uint64_t media_offset[HBF_MAX_RANGES];
    uint32_t perms[HBF_MAX_RANGES];
    uint32_t count;
    uint32_t pad;
};

// Exact unsigned division of n < 2^63 by a run-time constant: one multiply-high and a shift.
struct Div64 { uint64_t magic; uint32_t shift; uint32_t pow2; };

// Geometry and timing, fixed at create.
struct ModelParams {
    uint32_t channels, dies, planes;
    uint32_t n_queues, n_dies;
    uint32_t page_shift, stripe_shift, pages_per_stripe_shift;
    uint32_t queue_level;
    uint32_t pow2_geom;                  // channels, dies, planes all powers of two
    uint32_t ch_shift, die_shift, plane_shift;
    uint32_t read_gran_shift, prog_gran_shift;
    int64_t t_read_ns, t_prog_ns;
    uint64_t chan_bytes_per_us;
    Div64 div_chan;                      // division by chan_bytes_per_us
    const uint32_t *xfer_tab;            // device: transfer ns of charged bytes k << xfer_tab_shift, k = 0..1024
    uint32_t xfer_tab_shift, xfer_tab_max_cb;
    int64_t e_cmd_read_pj, e_byte_read_pj, e_cmd_prog_pj, e_byte_prog_pj;
};

// Radix plan of one batch, written by the plan kernel.
struct SortPlan {
    uint32_t n_passes;
    uint32_t lo_bits, hi_bits;           // participating bits of the issue field and of the queue field
    uint32_t shift[kMaxPasses];
    uint32_t bits[kMaxPasses];
};

// Per-batch control block in device memory, cleared by the begin kernel.
struct BatchCtrl {
    int32_t code;                        // HBF_OK or the batch's refusal / failure code
    int32_t skip;                        // later kernels do nothing when set
    int32_t mode; int32_t pad0;
    int64_t q_ppm;
    Div64 div_q;                         // division by the batch's snapshot of q
    unsigned long long n_native, n_ready, n_fault;
    unsigned long long key_or, key_and;
    uint32_t unsorted;                   // some record has a smaller issue time than its predecessor
    uint32_t inorder_used;               // the in-order path served this batch
    uint32_t run_sort;                   // the sort path has to serve this batch
    uint32_t pad1;
    uint32_t role_count[2];              // in-order serve pass: tiles handed out so far, per size class
    uint32_t tile_counter[kMaxPasses + 2];
    long long modeled_ns, service_ns, max_completion_ns;
    SortPlan plan;
};

// Long-lived device state of a context.
struct DevState {
    int32_t mode; int32_t poisoned;
    int64_t q_ppm;
    uint32_t spin_limit;                 // polls of one look-back slot before a waiter gives up (kSpinLimit unless a test lowers it)
    uint32_t test_stage, test_tile;      // test support: tile `test_tile` of stage 1 (first radix pass) or 2 (scan) publishes nothing
    uint32_t pad;
};

// Workspace carve-up for a batch of n records.
struct Workspace {
    uint64_t *keys[2];
    uint32_t *idx[2];
    uint64_t *terms;                     // [n] per record, in batch order: bytes | op << 32 | pages << 33 (what the scan needs of it)
    uint32_t *hist;                      // [kMaxPasses][kRadix]
    uint32_t *sort_desc[2];              // [tiles][kRadix] look-back words, ping-pong between passes
    void *scan_desc;                     // [scan tiles] ScanDesc
    int64_t *in_agg;                     // [tiles][queues][2]: per-tile, per-queue max-plus aggregate (S, M)
    int64_t *in_bin;                     // [tiles][queues]: busy-until entering each tile
    void *in_tile;                       // [tiles] stall bookkeeping of the in-order path
    void *in_head;                       // [tiles]: the first 8 accesses of every (tile, queue) for the fix-up: a tile's first entries, then each queue's other seven
    uint8_t *in_headcnt;                 // [tiles][queues]: how many of them exist; 0xff marks a queue for the straggle pass
    uint16_t *in_qid;                    // [tiles][stride]: queue of each of the first records of every tile (0xffff: not modeled), for the straggle pass
    uint32_t *bus_xfer;                  // [n] transfer time of every read (only with the channel-bus stage on)
    size_t bytes;
};

// The registered ranges when there is exactly one of them (on == 0 otherwise): what the in-order kernels take as
// a kernel argument, so that the common configuration reads nothing from memory to classify an access.
struct FastRange { uint64_t base, length, media_offset; uint32_t perms, on; };

struct TileBalanceHost;
struct SubmitArgs {
    const hbf_access_t *acc; uint64_t n;
    int64_t *completion, *stall; uint8_t *status; hbf_die_stats_t *die_stats;
    const RangeSnap *ranges; const ModelParams *mp_dev; ModelParams mp;
    DevState *state; BatchCtrl *ctrl; hbf_batch_result_t *result;
    int64_t *busy, *busy_stage, *pending; hbf_die_stats_t *stats_stage;
    Workspace ws; int32_t path; int sm_count; int inorder_ok;
    FastRange fast;
    int binned;                          // the batch's energy goes to the time-bin ledger, not to the pending totals
    int bus_on;                          // the channel-bus stage follows: array-done times must fit its 47-bit key field
    const unsigned long long *claim_limit;  // retention on: batch index below which a modeled access claims a refresh quantum
    uint32_t *die_claims;                   // retention on: [dies] claims of the batch
    const struct RetDev *ret;               // retention on: the block state (host copy of the device pointers)
    cudaEvent_t *ev;                     // [kProfEvents] or null: recorded between kernel groups
    TileBalanceHost *bal;                // tile sizes from measurements (null: off)
};
constexpr int kProfEvents = 10;
extern std::atomic<unsigned long long> g_kernel_launches;
// The dynamic shared memory a kernel may use is an attribute of the (device, kernel) pair: raises it on the current device
// when `bytes` exceeds what this process has set there so far.  Thread-safe.
cudaError_t ensure_dyn_smem(const void *kernel, size_t bytes);

constexpr uint32_t kInMaxQueues = 2048;  // the in-order path keeps per-queue state in shared memory
constexpr uint32_t kInMaxTiles = 1024;
constexpr uint32_t kInTileQuantum = 1024; // tiles of the in-order path are a multiple of this many records
constexpr uint32_t kInQidPrefix = 131072; // records at the head of a tile whose queue numbers the serve pass leaves for the straggle pass
// 16-bit queue numbers kept for a batch of n records (an upper bound over every tiling of it)
inline uint64_t inorder_qid_entries(uint64_t n) {
    const uint64_t a = 2 * (n + kInTileQuantum), b = (uint64_t)kInMaxTiles * kInQidPrefix;
    return a < b ? a : b;
}
// upper bound of the number of tiles of a batch of n records, on any device: what the workspace is carved for
inline uint64_t inorder_tiles_bound(uint64_t n) {
    const uint64_t t = (n + kInTileQuantum - 1) / kInTileQuantum;
    return t < 1 ? 1 : (t < kInMaxTiles ? t : kInMaxTiles);
}
size_t workspace_layout(uint64_t n, uint32_t n_queues, Workspace *ws, void *base, int with_bus = 0);
// channel bus as a second queued stage, after launch_submit on the same arguments (bc: a control block of its own)
cudaError_t launch_bus_stage(const SubmitArgs &a, BatchCtrl *bc, int64_t *bus_busy, cudaStream_t st);
// How the in-order path cuts a batch of n records into contiguous tiles: n_big tiles of `big` records, then tiles of
// `small` records (the last one ragged).  All sizes are multiples of kInTileQuantum.  n_big == 0: one size only.
// With `first` set (device memory, n_tiles + 1 entries) the tiles begin where that table says instead: sizes that follow
// from how long each tile's block took in an earlier batch (TileBalance below).  by_sm: a block takes the tile of its SM
// and of its kind (tile = kind * n_big + SM), so that a tile's time tells how fast that place serves.
struct InTileMap { uint64_t n; uint32_t n_tiles, n_big; uint32_t big, small; const uint32_t *first; uint32_t max_tile, by_sm; };
__device__ inline uint64_t tile_first(const InTileMap &m, uint32_t t) {
    if (m.first) return m.first[t];
    return t < m.n_big ? (uint64_t)t * m.big : (uint64_t)m.n_big * m.big + (uint64_t)(t - m.n_big) * m.small;
}
__device__ inline uint64_t tile_last(const InTileMap &m, uint32_t t) {      // one past the tile's last record
    const uint64_t e = m.first ? (uint64_t)m.first[t + 1] : tile_first(m, t) + (t < m.n_big ? m.big : m.small);
    return e < m.n ? e : m.n;
}
// Tile sizes from measurements.  The SMs of a device do not serve a tile equally fast (the same few are about 3 % slower
// in every launch, and of the two blocks of an SM the one in the lower warp slots is faster), and the pass lasts as long
// as its slowest block.  Every block of the streaming pass leaves how many records its tile had and how long it took;
// the host reads that record of an earlier batch (an asynchronous copy: nothing waits for it) and sizes the next
// batch's tiles in proportion to the measured rates.  Results do not depend on where tiles begin.
constexpr uint32_t kInBalMax = 320;      // tiles this can describe (two per SM)
struct TileBalance {
    uint32_t claim[kInBalMax];           // number of the last batch in which the tile was taken (hand-out by SM and kind)
    uint32_t len[kInBalMax], ns[kInBalMax];   // records of the tile, and how long its block took (0: taken out of turn, not measured)
    uint32_t strag_seq, strag_max, strag_flagged, strag_depth;   // of batch strag_seq: most straggling queues in a tile, tiles served a second time, head entries kept
    uint32_t first[kInBalMax + 1];       // device only: where the tiles of the batch in flight begin
};
struct TileBalanceHost { TileBalance *dev = nullptr, *pinned = nullptr; uint32_t seq = 0; bool on = true; uint32_t depth = 0, depth_fixed = 0, depth_seen = 0; };   // depth: head entries per (tile, queue) of the next batch (0: the most); depth_fixed != 0: set by the caller; depth_seen: batch whose record was read last
InTileMap inorder_tile_map(uint64_t n, int sm_count, bool by_table);   // by_table: a full wave gets exactly two tiles per SM, placed by a table
// per-tile bookkeeping of the stall total: as-if-idle sum, fix-up corrections, and the exact sum of a re-served tile
struct InTile { long long spec_sum, fix_delta, true_sum; uint32_t reserve; uint32_t stragglers; };
size_t inorder_head_bytes(uint64_t tiles, uint32_t n_queues);
size_t inorder_serve_smem(uint32_t n_dies);
cudaError_t launch_inorder(const SubmitArgs &a, cudaStream_t st);
constexpr uint32_t kInSmallMax = 8192;   // batches of at most this many records are served by one block in one launch
bool inorder_small_batch(uint64_t n);   // whether launch_inorder takes that route
uint32_t inorder_small_blocks(uint32_t n_queues);   // its blocks: each leaves one entry of the tile table (the slice's stall total)
cudaError_t launch_submit(const SubmitArgs &a, cudaStream_t st);
// total[i] += part[i] over the 6 * n_dies counters of a per-die statistics array (host-buffer pipeline: totals over its chunks)
cudaError_t launch_add_stats(hbf_die_stats_t *total, const hbf_die_stats_t *part, uint32_t n_dies, cudaStream_t st);
// the same for batch summaries: counts and times added, the largest completion, the first code that is not HBF_OK; first != 0 starts over
cudaError_t launch_add_result(hbf_batch_result_t *sum, const hbf_batch_result_t *part, int first, cudaStream_t st);
cudaError_t launch_queue_order(const BatchCtrl *ctrl, const Workspace &ws, uint32_t *out, uint64_t n, cudaStream_t st);

// ---- page-granular submit ---------------------------------------------------------------------------
struct PagedWorkspace {
    unsigned long long *tile_sum;        // [tiles of 2,048 accesses] parts per tile, then exclusive offsets
    uint32_t *row_off;                   // [rows of 32 accesses] parts before the row within its tile
    unsigned long long *total;           // parts of the batch
    void *sums;                          // accesses served and their stall total
    uint32_t *part_first;                // [n + 1] first part of every access
    hbf_access_t *parts;                 // [capacity] the parts as access records
    int64_t *part_completion, *part_stall; uint8_t *part_status;
    void *inner; size_t inner_bytes;     // workspace of the ordinary path for `capacity` records
    size_t bytes;
};
size_t paged_layout(uint64_t n, uint64_t capacity, uint32_t n_queues, PagedWorkspace *pw, void *base, int with_bus = 0);
cudaError_t launch_paged_count(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev,
                               const PagedWorkspace &pw, cudaStream_t st);
cudaError_t launch_paged_expand(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev,
                                const FastRange &fast, uint32_t page_shift, uint64_t capacity, const PagedWorkspace &pw, int sm_count,
                                cudaStream_t st);
cudaError_t launch_paged_join(const hbf_access_t *acc, uint64_t n, const PagedWorkspace &pw, hbf_batch_result_t *result,
                              int64_t *completion, int64_t *stall, uint8_t *status, int sm_count, cudaStream_t st);

// ---- time-bin energy ledger ----------------------------------------------------------------------------
cudaError_t launch_energy_bins(const hbf_access_t *acc, uint64_t n, const int64_t *completion, const RangeSnap *ranges,
                               const ModelParams *mp_dev, const BatchCtrl *ctrl, const hbf_batch_result_t *result,
                               unsigned long long *ledger, int64_t bin_ns, uint32_t n_bins, int64_t cur_bin, int sm_count,
                               const unsigned long long *claim_limit, int64_t quantum_pj, cudaStream_t st);
cudaError_t launch_take_bin(unsigned long long *row, int64_t *pending, uint32_t n_dies, cudaStream_t st);

// ---- reduced-order thermal model -------------------------------------------------------------------------
cudaError_t launch_rom_steps(uint32_t n, uint32_t m, uint32_t o, const double *A, const double *B, const double *b,
                             const double *C, const double *D, const double *d, double *x, const double *power,
                             uint32_t n_steps, double *temps_out, cudaStream_t st);

// ---- retention, refresh and wear (Design D4) -------------------------------------------------------------
// Device-resident counters of the refresh plan.  planned - claimed - decayed quanta are outstanding (the debt).
struct RetState {
    unsigned long long planned, claimed, decayed, commits, worn_blocks;
    unsigned long long claim_limit;      // this batch: modeled accesses with a smaller batch index claim one quantum each
    unsigned long long claims_now;       // quanta this batch claims if it is accepted
    unsigned long long tickets, counted; // the claim window's tile counter and the modeled accesses counted so far
    unsigned long long epoch_total;      // quanta the epoch in progress adds
    uint32_t epoch;
    uint32_t observed_inline;            // the in-order serve pass has counted this batch's reads into the disturb counters
};
constexpr uint32_t kRetTabChannels = 128;
struct RetDev {
    uint32_t ppb, bpp, bpz, max_pec, disturb_limit, n_regions;
    Div64 div_ppb, div_bpp;              // exact division by pages_per_block and by blocks_per_plane
    uint32_t pow2, ppb_shift;            // pages_per_block and blocks_per_plane are powers of two (and a plane has fewer than 2^32 pages): shifts do
    double accel, lead, l_ref_s, t_ref_k, ea_over_kb;
    uint64_t n_blocks, plan_cap;
    double *damage; uint32_t *disturb, *pec, *epoch_of; uint8_t *worn;
    unsigned long long *last_pos;        // [blocks] plan position of the block's last quantum
    uint32_t *plan;                      // [plan_cap] ring of quanta (block * ppb + page), position modulo plan_cap
    uint32_t *rank;                      // [blocks] rank of a newly eligible block in its die's (zone, plane, block) order
    unsigned long long *die_len, *chan_len;   // quanta the epoch in progress adds per die, per channel
    uint32_t *chan_tab;                  // the channels' lengths sorted, their running sums, and per channel the sorted lengths of the channels before it (null: more than kRetTabChannels channels)
    uint32_t *die_claims;                // [dies] quanta claimed on each die by the batch in progress
    uint32_t *tile_count;                // [tiles of 1,024 records] modeled accesses, claim window
    double *rate, *region_temp;          // [regions] damage per block of this epoch; temperatures
    int *region_max;                     // [regions] hottest cell, as an ordered integer
    RetState *st;
};
cudaError_t launch_ret_window(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const RetDev &r, int sm_count, cudaStream_t st);
cudaError_t launch_ret_close(const hbf_access_t *acc, uint64_t n, const RangeSnap *ranges, const ModelParams *mp_dev, const ModelParams &mp,
                             const hbf_batch_result_t *result, int64_t *pending, int binned, const RetDev &r, int sm_count, cudaStream_t st);
struct ThermalDev;
cudaError_t launch_ret_advance(const RetDev &r, const ModelParams &mp, const ThermalDev *field, const float *theta, const int32_t *die_region,
                               int have_temps, int64_t dt_ns, int sm_count, cudaStream_t st);
cudaError_t launch_ret_decay(const RetDev &r, const ModelParams &mp, const DevState *state, int64_t idle_ns, int sm_count, cudaStream_t st);

// ---- thermal -------------------------------------------------------------------------------------
struct ThermalDev {
    uint32_t H, W, n_regions, n_dies, n_sub;
    float ambient_c;
    int64_t rtt_mk, ltt_mk, stt_mk, shut_mk, q_light_ppm;
    const float *C, *Gx, *Gy, *Gs;
    const int32_t *cell_region, *die_region, *region_kind;
    const float *region_idle_w; const float *region_inv_cells;
    const int32_t *region_die_ptr, *region_die_list;   // dies of each region, CSR
    float *theta[2]; float *comp; float *P; double *region_power; float *ext_power;
    float *hot;                          // [3] device
};
cudaError_t launch_thermal_step(const ThermalDev &t, DevState *state, int64_t *pending, int64_t dt_ns,
                                int has_ext, float *d_temps_out, int *cur, int generic_only, cudaStream_t st);

cudaError_t launch_rom_power(const ThermalDev &t, int64_t *pending, int64_t dt_ns, int has_ext, double *p_out, cudaStream_t st);
cudaError_t launch_rom_controller(const ThermalDev &t, const double *temps, const int32_t *kind, uint32_t n_out, DevState *state,
                                  cudaStream_t st);

}  // namespace hbf
