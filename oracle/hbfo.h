/*
 * hbfo -- sequential CPU oracle of the HBF service model.  TEST INFRASTRUCTURE ONLY.
 *
 * This is the plain definition of what the GPU library computes, one access at a time, written
 * from the paper (HBFSim) and from the stated readings of what the paper leaves open.  It shares
 * no code, header, table or helper with the CUDA path.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the product path never does.
 *
 * What follows the paper directly:
 *   - range classification, fail-closed            (Design D1, "An Explicit and Fail-Closed Boundary")
 *   - ticket = slot index, result lands at the same index   (Implementation, control region)
 *   - thermal service scaling s_T = ceil(s*10^6/q)  (Eq. 3)
 *   - throttle modes Normal/Light/Severe/Shutdown   (Design D3)
 *   - event energy E = E_command + e_byte*bytes, P = E/dt + P_idle   (Design D3)
 *   - RC node equation                              (Eq. 1)
 * What is a reading (the paper gives no equations for the queue itself, no plane/die timing and
 * no threshold values): the FIFO recurrence start = max(arrival, busy_until), the address
 * interleave, data transfer as pure latency, granule rounding, the threshold numbers.
 *
 * Pins: hand-worked single-queue examples, the closed form n*tR + transfer, queue invariants,
 * an independent event-driven brute force on tiny inputs, the M/D/1 mean wait, the printed power
 * figure 37.256 W at 384 GB/s, thermal steady state against a direct linear solve and the lumped
 * closed form.  Parity unpinned (no value in the paper, fixed by the committed profile only):
 * program energy per byte, the threshold temperatures, q_light, the floorplan constants; of the retention part
 * (Design D4) everything beyond the two equations, the eligibility rule, the emission order and the claim rule:
 * the block layout, the cost and the booking of a quantum, the read-disturb increment, when a commit takes effect,
 * the decay rate (pinned against hand-worked examples of this build's own definitions only).
 *
 * All times int64 ns on one shared origin; energies int64 pJ; temperatures double, deg C.
 */
#ifndef HBFO_H
#define HBFO_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { HBFO_OK = 0, HBFO_E_INVAL = -1, HBFO_E_RANGE_OVERLAP = -2, HBFO_E_RANGE_FULL = -3,
       HBFO_E_CAPACITY = -4, HBFO_E_WORKSPACE = -5, HBFO_E_CUDA = -6, HBFO_E_ACCESS_FAULT = -7,
       HBFO_E_THROTTLED = -8, HBFO_E_LINK_SHUTDOWN = -9, HBFO_E_TIMEOUT = -10, HBFO_E_NOMEM = -11 };
enum { HBFO_ST_NATIVE = 0, HBFO_ST_READY = 1, HBFO_ST_FAULT_PARTIAL = 2, HBFO_ST_FAULT_PERM = 3,
       HBFO_ST_UNSUPPORTED = 4 };
enum { HBFO_MODE_NORMAL = 0, HBFO_MODE_LIGHT = 1, HBFO_MODE_SEVERE = 2, HBFO_MODE_SHUTDOWN = 3 };
enum { HBFO_KIND_NONE = 0, HBFO_KIND_GPU = 1, HBFO_KIND_HBM = 2, HBFO_KIND_HBF = 3 };
#define HBFO_MAX_RANGES 64

typedef struct { uint64_t addr; int64_t issue_ns; uint32_t bytes; uint32_t flags; } hbfo_access_t;
typedef struct { int64_t busy_ns, bytes_read, bytes_prog, energy_pj, n_read, n_prog; } hbfo_die_stats_t;
typedef struct {
    int32_t code, mode; int64_t q_ppm; uint64_t n_native, n_modeled, n_fault;
    int64_t modeled_ns, service_ns, max_completion_ns;
} hbfo_batch_result_t;

typedef struct {
    uint32_t channels, dies, planes, page_bytes, stripe_bytes, queue_level;
    uint64_t capacity_bytes;
    int64_t  t_read_ns, t_prog_ns;
    uint64_t chan_bytes_per_us;
    uint32_t read_granule, prog_granule;
    int64_t  e_cmd_read_pj, e_byte_read_pj, e_cmd_prog_pj, e_byte_prog_pj;
    uint32_t grid_h, grid_w, n_sub, n_regions;
    float    ambient_c, rtt_c, ltt_c, stt_c, shutdown_c;
    int64_t  q_light_ppm;
    const float *cell_C, *cell_Gx, *cell_Gy, *cell_Gsink;      /* [grid_h*grid_w]; NULL cell_C => no thermal */
    const int32_t *cell_region;                                /* [grid_h*grid_w], -1 = no region */
    const int32_t *die_region;                                 /* [channels*dies] */
    const int32_t *region_kind;                                /* [n_regions] */
    const float *region_idle_w;                                /* [n_regions] */
} hbfo_config_t;

typedef struct hbfo_ctx hbfo_ctx;

int  hbfo_create(const hbfo_config_t *cfg, hbfo_ctx **out);
int  hbfo_destroy(hbfo_ctx *ctx);
int  hbfo_register_range(hbfo_ctx *ctx, uint64_t base, uint64_t length, uint32_t perms, uint32_t kind,
                         uint32_t stream_tag, uint64_t media_offset, uint32_t *out_id);
int  hbfo_clear_ranges(hbfo_ctx *ctx);
int  hbfo_submit_batch(hbfo_ctx *ctx, const hbfo_access_t *acc, uint64_t n, int64_t *completion_ns,
                       int64_t *stall_ns, uint8_t *status, hbfo_die_stats_t *die_stats);
/* Page-granular variant (this build's extension; the paper's back end is a page-based flash simulator but the
 * text does not spell the splitting out): every page of a modeled access is a request of its own, queued by
 * its own decode; the access completes with its last part.  Same arguments as hbfo_submit_batch.  The parts, listed
 * in (access, part) order, are served as hbfo_submit_batch serves a batch of accesses, so the energy bins, the
 * channel bus and retention, when on, see parts: one ledger event, one bus transfer, one possible refresh claim and
 * one disturbing read per part. */
int  hbfo_submit_batch_paged(hbfo_ctx *ctx, const hbfo_access_t *acc, uint64_t n, int64_t *completion_ns,
                             int64_t *stall_ns, uint8_t *status, hbfo_die_stats_t *die_stats);
/* Time-bin power integration (Section "Design", event-based energy model: a ledger of energy per time bin, a long
 * event shared among its bins by time spent in each).  After this call hbfo_submit_batch books every access's
 * energy into the bins its array service interval overlaps instead of the pending total, and
 * hbfo_thermal_step(dt_ns == bin_ns) consumes the bin the thermal clock stands in.  hbfo_get_energy_bins
 * copies the ring out, row k = bin first_bin + k.  hbfo_reset clears the ring and the clock. */
int  hbfo_enable_energy_bins(hbfo_ctx *ctx, int64_t bin_ns, uint32_t n_bins);
int  hbfo_get_energy_bins(hbfo_ctx *ctx, int64_t *out, uint64_t cap, int64_t *first_bin);
/* Channel bus as a second queued stage (this build's extension): after this call a read's data-out transfer
 * queues on its channel's bus in (array-done time, batch index) order instead of being a fixed latency; programs
 * are unchanged.  hbfo_get_bus_busy_until copies the per-channel bus state out.  hbfo_reset clears it. */
int  hbfo_enable_channel_bus(hbfo_ctx *ctx);
int  hbfo_get_bus_busy_until(hbfo_ctx *ctx, int64_t *out, uint64_t cap);
int  hbfo_last_result(hbfo_ctx *ctx, hbfo_batch_result_t *out);
/* The order in which the last accepted batch was served: indices, queue-major. */
int  hbfo_last_order(hbfo_ctx *ctx, uint32_t *order, uint64_t cap, uint64_t *count);
int  hbfo_thermal_step(hbfo_ctx *ctx, int64_t dt_ns, const float *ext_power_w, uint32_t n_ext,
                       double *temps_out, double hot_c_out[3]);
int  hbfo_force_mode(hbfo_ctx *ctx, int32_t mode, int64_t q_ppm);
int  hbfo_reset(hbfo_ctx *ctx);
/* State readers/writers used by tests. */
int  hbfo_get_busy_until(hbfo_ctx *ctx, int64_t *out, uint64_t cap);
int  hbfo_get_pending_energy(hbfo_ctx *ctx, int64_t *out, uint64_t cap);
int  hbfo_get_temps(hbfo_ctx *ctx, double *out, uint64_t cap);
int  hbfo_set_temps(hbfo_ctx *ctx, const double *in, uint64_t count);
int  hbfo_get_mode(hbfo_ctx *ctx, int32_t *mode, int64_t *q_ppm);
double hbfo_euler_limit_ns(hbfo_ctx *ctx);
/* Single steps of the definition, exposed so that each can be pinned on its own. */
int  hbfo_classify(hbfo_ctx *ctx, const hbfo_access_t *a, int32_t *range_id);
int  hbfo_decode(hbfo_ctx *ctx, uint64_t off, uint32_t bytes, uint32_t *channel, uint32_t *die,
                 uint32_t *plane, uint64_t *row, uint64_t *page, uint64_t *npages, uint32_t *queue);
int  hbfo_service_terms(hbfo_ctx *ctx, uint32_t bytes, uint64_t npages, uint32_t op, int64_t q_ppm,
                        int64_t *charged_bytes, int64_t *xfer_ns, int64_t *s_ns, int64_t *energy_pj);
int32_t hbfo_next_mode(hbfo_ctx *ctx, int32_t mode, int64_t t_hot_mk);
int64_t hbfo_quantise_mk(double t_c);
const char *hbfo_strerror(int code);

/* Retention, refresh and wear (Design D4; the definitions and the readings are at the head of this part of
 * hbfo.c).  Not together with the page-granular submit; with the energy bins on, a claimed
 * quantum is booked as an event of its own ahead of the claiming access's.
 *   hbfo_enable_retention     block state for channels*dies*planes*blocks_per_plane blocks, all fresh
 *   hbfo_retention_advance    one epoch: damage += accel*dt/L(T) per block with its die's region temperature
 *                             (region_temp_c [n_regions], or NULL = hottest cell of each region in the field),
 *                             newly eligible blocks join the plan in the deterministic order
 *   hbfo_submit_batch         the modeled accesses claim the outstanding quanta in index order, one each; reads
 *                             count towards read disturb; blocks whose quanta are all claimed commit
 *   hbfo_retention_decay      idle time drains outstanding quanta, one per scaled quantum time */
typedef struct {
    uint32_t pages_per_block, blocks_per_plane, blocks_per_zone;
    uint32_t max_pec;                      /* a block that has committed this many cycles is worn out */
    uint32_t disturb_limit;                /* page reads that make a block eligible; 0 = no limit */
    uint32_t pad;
    double l_ref_s, t_ref_c, ea_ev;        /* lifetime at the reference temperature; activation energy */
    double accel;                          /* a_t, reliability-time acceleration */
    double lead_threshold;                 /* damage at which a block becomes eligible */
} hbfo_retention_config_t;
typedef struct {
    uint64_t n_blocks, planned, claimed, decayed, commits, worn_blocks, waiting_blocks;
    uint32_t epoch, pad;
} hbfo_retention_totals_t;
int  hbfo_enable_retention(hbfo_ctx *ctx, const hbfo_retention_config_t *cfg);
int  hbfo_retention_advance(hbfo_ctx *ctx, int64_t dt_ns, const double *region_temp_c);
int  hbfo_retention_decay(hbfo_ctx *ctx, int64_t idle_ns);
int  hbfo_get_retention_blocks(hbfo_ctx *ctx, double *damage, uint32_t *disturb, uint32_t *pec, uint32_t *epoch, uint64_t cap);
/* the outstanding quanta in plan order (quantum = block * pages_per_block + page); quanta == NULL: count only */
int  hbfo_get_retention_plan(hbfo_ctx *ctx, uint32_t *quanta, uint64_t cap, uint64_t *count);
int  hbfo_get_retention_totals(hbfo_ctx *ctx, hbfo_retention_totals_t *out);
double hbfo_retention_lifetime_s(hbfo_ctx *ctx, double temp_c);

/* Reduced-order thermal model (Eq. 2): x' = A x + B p + b, T = C x + D p + d (x before the update).  Matrices
 * row-major, double, copied at create; b, D, d may be NULL (zero).  The state starts at zero. */
typedef struct hbfo_rom hbfo_rom;
int  hbfo_rom_create(uint32_t n_states, uint32_t n_inputs, uint32_t n_outputs, const double *A, const double *B,
                     const double *b, const double *C, const double *D, const double *d, hbfo_rom **out);
int  hbfo_rom_destroy(hbfo_rom *rom);
int  hbfo_rom_reset(hbfo_rom *rom);
int  hbfo_rom_step(hbfo_rom *rom, const double *power, uint32_t n_steps, double *temps_out);
int  hbfo_rom_get_state(hbfo_rom *rom, double *out, uint64_t cap);

/* One thermal step on the reduced-order model instead of the grid: the same power vector (one entry per region),
 * one model step, the controller on the hottest output of each medium (output_kind[i] = HBFO_KIND_* of output i). */
int  hbfo_thermal_step_rom(hbfo_ctx *ctx, hbfo_rom *rom, const int32_t *output_kind, int64_t dt_ns,
                           const float *ext_power_w, uint32_t n_ext, double hot_c_out[3]);

#ifdef __cplusplus
}
#endif
#endif
