/*
 * hbf.h -- C ABI of the B200 HBF service-model library (libhbf.so).
 *
 * The library applies an online High-Bandwidth-Flash service model to batches of memory accesses:
 * range check, address decode to channel/die/plane/page, per-queue FIFO service, completion time
 * and injected stall per access, per-die busy/byte/energy totals, and the coupled package thermal
 * step with its throttle controller.  Every step runs in CUDA kernels (sm_100a); there is no CPU
 * path.  "device" pointers are CUDA device memory owned by the caller; "host" pointers are plain
 * host memory.  All times are int64 ns on one caller-chosen origin (the paper forbids mixing clock
 * origins, Design D3); energies are int64 pJ; temperatures are float degrees C.
 *
 * Return values: 0 = HBF_OK, negative = error.  Nothing is downgraded silently (Implementation,
 * "Every failure ends the run").  Calls on one context must come from one thread at a time.  A context
 * belongs to the CUDA device that was current at hbf_create: hbf_submit_batch, hbf_submit_batch_paged and
 * hbf_thermal_step return HBF_E_INVAL when another device is current.
 */
#ifndef HBF_H
#define HBF_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define HBF_API __attribute__((visibility("default")))
#else
#define HBF_API
#endif

enum {
    HBF_OK = 0,
    HBF_E_INVAL = -1,          /* null pointer, zero size, non-power-of-two page/stripe/granule, bad mode ... */
    HBF_E_RANGE_OVERLAP = -2,  /* overlapping registration would make classification ambiguous (Design D1) */
    HBF_E_RANGE_FULL = -3,     /* more than HBF_MAX_RANGES ranges */
    HBF_E_CAPACITY = -4,       /* media_offset + length beyond capacity_bytes */
    HBF_E_WORKSPACE = -5,      /* workspace smaller than hbf_workspace_bytes(n) or misaligned */
    HBF_E_CUDA = -6,           /* a CUDA runtime call failed */
    HBF_E_ACCESS_FAULT = -7,   /* >= 1 fail-closed access: batch refused, status[] filled, outputs zeroed, no state change */
    HBF_E_THROTTLED = -8,      /* mode Severe: new reservations withheld, no state change (Design D3) */
    HBF_E_LINK_SHUTDOWN = -9,  /* mode Shutdown: terminal, every later batch returns it (Design D3) */
    HBF_E_TIMEOUT = -10,       /* a bounded device-side wait expired; the context is poisoned */
    HBF_E_NOMEM = -11
};

/* Per-access status: the batch analogue of the paper's per-request terminal states (Implementation). */
enum { HBF_ST_NATIVE = 0,        /* address outside every range: native HBM path, not modeled */
       HBF_ST_READY = 1,         /* whole span inside one range and permitted: modeled */
       HBF_ST_FAULT_PARTIAL = 2, /* starts inside a range but leaves it (or wraps) */
       HBF_ST_FAULT_PERM = 3,    /* operation not permitted by the range */
       HBF_ST_UNSUPPORTED = 4 }; /* bytes == 0, unknown flag bits, issue_ns < 0; also issue_ns >= HBF_ISSUE_LIMIT (see there) */

enum { HBF_MODE_NORMAL = 0, HBF_MODE_LIGHT = 1, HBF_MODE_SEVERE = 2, HBF_MODE_SHUTDOWN = 3 };
enum { HBF_KIND_NONE = 0, HBF_KIND_GPU = 1, HBF_KIND_HBM = 2, HBF_KIND_HBF = 3 };     /* region kinds */
enum { HBF_PERM_READ = 1, HBF_PERM_PROGRAM = 2 };
enum { HBF_RANGE_TIMING = 0, HBF_RANGE_CAPACITY = 1 };
enum { HBF_PATH_AUTO = 0, HBF_PATH_SORT = 1, HBF_PATH_INORDER = 2, HBF_PATH_SORT_FULL = 3 };

#define HBF_MAX_RANGES 64
#define HBF_MAX_BATCH ((uint64_t)((1u << 30) - 1))      /* accesses per batch */
/* A restriction of this library, not of the model: the sort path packs (queue, issue_ns) into one 64-bit key with 47 bits
 * for the issue time, so an access with issue_ns >= 2^47 (39 h on the caller's clock; the paper's longest run is 86,400 s)
 * is marked HBF_ST_UNSUPPORTED and its batch is refused with HBF_E_ACCESS_FAULT, nothing changed.  The model itself has
 * no such bound; a caller with later times moves its clock origin. */
#define HBF_ISSUE_LIMIT (((int64_t)1) << 47)

/* One access record, 24 bytes.  flags bit 0: 0 = read, 1 = program; all other bits must be 0. */
typedef struct { uint64_t addr; int64_t issue_ns; uint32_t bytes; uint32_t flags; } hbf_access_t;

/* Per-die totals of one batch ([channels*dies], index channel*dies + die). */
typedef struct { int64_t busy_ns, bytes_read, bytes_prog, energy_pj, n_read, n_prog; } hbf_die_stats_t;

/* Batch summary.  modeled_ns = sum of stalls, service_ns = sum of queue service: two of the paper's
 * four time counters (Implementation); the other two are wall-clock quantities of the caller. */
typedef struct {
    int32_t code, mode; int64_t q_ppm; uint64_t n_native, n_modeled, n_fault;
    int64_t modeled_ns, service_ns, max_completion_ns;
} hbf_batch_result_t;

typedef struct {
    /* geometry: a media offset is striped channel first, then die, then plane, in units of stripe_bytes */
    uint32_t channels, dies, planes, page_bytes, stripe_bytes;
    uint32_t queue_level;                 /* 0: one queue per plane, 1: one queue per die */
    uint64_t capacity_bytes;              /* 0 = unbounded */
    /* timing */
    int64_t  t_read_ns, t_prog_ns;        /* array time per page */
    uint64_t chan_bytes_per_us;           /* data transfer rate of one channel */
    uint32_t read_granule, prog_granule;  /* charged bytes are rounded up to these (powers of two) */
    /* energy: E = e_cmd + e_byte * charged bytes (Design D3) */
    int64_t  e_cmd_read_pj, e_byte_read_pj, e_cmd_prog_pj, e_byte_prog_pj;
    /* thermal (ignored when cell_C is NULL) */
    uint32_t grid_h, grid_w, n_sub, n_regions;
    float    ambient_c, rtt_c, ltt_c, stt_c, shutdown_c;   /* rtt < ltt < stt < shutdown */
    int64_t  q_light_ppm;                 /* service fraction published in Light mode, 1..10^6 */
    const float *cell_C, *cell_Gx, *cell_Gy, *cell_Gsink;  /* host [grid_h*grid_w]; Gx[y][x] joins (y,x),(y,x+1); Gy[y][x] joins (y,x),(y+1,x) */
    const int32_t *cell_region;           /* host [grid_h*grid_w], -1 = cell belongs to no region */
    const int32_t *die_region;            /* host [channels*dies] -> region */
    const int32_t *region_kind;           /* host [n_regions], HBF_KIND_* */
    const float *region_idle_w;           /* host [n_regions] */
} hbf_config_t;

typedef struct hbf_ctx hbf_ctx;           /* opaque, library-owned */

/* Validates the configuration, copies every host array, allocates the context's device state on the
 * current CUDA device.  cuda_stream is a cudaStream_t (NULL = default stream); all work of the
 * context is ordered on it.  Queue state starts idle, the thermal field at ambient, mode Normal. */
HBF_API int hbf_create(const hbf_config_t *cfg, void *cuda_stream, hbf_ctx **out);
HBF_API int hbf_destroy(hbf_ctx *ctx);

/* Registers the address interval [base, base+length) as an HBF range (Design D1: base, length,
 * permissions, stream tag, backing offset) and publishes a new sorted snapshot for later batches.
 * media_offset is the range's first byte on the media.  out_id (nullable) receives the range id. */
HBF_API int hbf_register_range(hbf_ctx *ctx, uint64_t base, uint64_t length, uint32_t perms, uint32_t kind,
                       uint32_t stream_tag, uint64_t media_offset, uint32_t *out_id);
HBF_API int hbf_clear_ranges(hbf_ctx *ctx);

/* Bytes of device scratch hbf_submit_batch needs for a batch of n accesses (256-byte aligned). */
HBF_API size_t hbf_workspace_bytes(const hbf_ctx *ctx, uint64_t n);

/* Serves one batch, asynchronously on the context's stream.  For access i (its index plays the role
 * of the paper's ring ticket: results land at the same index):
 *   classify (Design D1) -> decode -> service terms (Eq. 3 with the batch's snapshot of q) ->
 *   FIFO per queue in (issue_ns, index) order after everything earlier batches left on the queue ->
 *   d_completion_ns[i], d_stall_ns[i] = completion - issue.  NATIVE rows: completion = issue, stall 0.
 * d_acc [n] device, read only, 8-byte aligned.  d_completion_ns, d_stall_ns [n] device.  d_status [n]
 * device, nullable.  d_die_stats [channels*dies] device, nullable, overwritten with this batch's totals.
 * d_workspace: device scratch of at least hbf_workspace_bytes(n), 256-byte aligned, must stay valid
 * until the batch has run.  The return value covers argument checks and launches only; the batch's
 * own outcome (access fault, throttled, shutdown, timeout) is read with hbf_last_result. */
HBF_API int hbf_submit_batch(hbf_ctx *ctx, const hbf_access_t *d_acc, uint64_t n, int64_t *d_completion_ns,
                     int64_t *d_stall_ns, uint8_t *d_status, hbf_die_stats_t *d_die_stats,
                     void *d_workspace, size_t workspace_bytes);

/* The same service for a batch that lives in HOST memory (no step of the method is defined by this call, so it cites
 * none: it is hbf_submit_batch behind a copy pipeline).  The batch is cut into chunks of `chunk` records (0 = a default
 * of 4 M); the copy-in of chunk k+1, the service of chunk k and the read-back of chunk k-1 run on three streams of
 * the library, so both directions of the link are busy while the kernels run.  Equivalent to one hbf_submit_batch per
 * chunk, in order: for records in issue order that is the same as one batch.
 * h_acc [n] host, read only; h_completion_ns, h_stall_ns [n] host; h_die_stats [channels*dies] host, nullable: totals
 * over the chunks.  Pinned host memory (cudaMallocHost / cudaHostRegister) makes the copies asynchronous and
 * overlapped; pageable memory works, slower.  The library owns the device buffers (two chunks of records and results,
 * one workspace), allocated at the first call and kept until hbf_destroy; a larger chunk reallocates them.
 * The call returns when every result is in the caller's buffers.  summary_out (host, nullable) receives the chunks'
 * summaries added up (counts and times summed, the largest completion, mode and q of the first chunk) with code =
 * the first chunk code that is not HBF_OK; that code is also the return value.  A refused chunk (fail-closed access,
 * throttled) leaves zeros in its part of the outputs and changes no state; later chunks are still served. */
HBF_API int hbf_submit_host(hbf_ctx *ctx, const hbf_access_t *h_acc, uint64_t n, int64_t *h_completion_ns,
                            int64_t *h_stall_ns, hbf_die_stats_t *h_die_stats, uint64_t chunk, hbf_batch_result_t *summary_out);

/* Page-granular variant of hbf_submit_batch (an extension: the paper's back end is a page-based flash simulator,
 * Section "Design", but the text does not define the splitting; this is the library's definition).  A modeled
 * access is cut at the page boundaries of the media; every part is a request of its own: decoded by its own
 * first byte (so consecutive pages follow the stripe interleave), charged one page of array time (Eq. 3) and
 * the transfer of its own bytes in whole granules, queued in (issue_ns, access index, part index) order.  The
 * access completes when its last part does; d_stall_ns[i] = completion - issue.  d_die_stats counts parts
 * (page operations); the batch summary read with hbf_last_result counts accesses.  An access that is not
 * modeled (native, or failing) is one part.  The list of parts, in (access, part) order, is served as hbf_submit_batch
 * serves a batch of accesses, so whatever else is switched on sees parts: with the energy bins a part's array interval
 * is a ledger event on the part's die; with the channel-bus stage a read part's transfer queues on the bus of the part's
 * channel in (array-done time, position in the list of parts) order; with retention the parts claim outstanding
 * refresh quanta in list order, one each, and a read part disturbs the block of its own page.
 * parts_capacity: upper bound, chosen by the caller, of the number of parts of the batch (at least n; e.g.
 * n * (largest access / page_bytes + 2)); it sizes the workspace, hbf_workspace_bytes_paged(ctx, n, capacity).
 * The call counts the parts on the device and waits for that count (one stream synchronisation) before it
 * launches the rest; with more parts than parts_capacity it returns HBF_E_WORKSPACE and nothing has changed.
 * Other arguments, ownership and error behaviour as for hbf_submit_batch.  hbf_queue_order afterwards refers
 * to parts, not accesses. */
HBF_API size_t hbf_workspace_bytes_paged(const hbf_ctx *ctx, uint64_t n, uint64_t parts_capacity);
HBF_API int hbf_submit_batch_paged(hbf_ctx *ctx, const hbf_access_t *d_acc, uint64_t n, uint64_t parts_capacity,
                           int64_t *d_completion_ns, int64_t *d_stall_ns, uint8_t *d_status,
                           hbf_die_stats_t *d_die_stats, void *d_workspace, size_t workspace_bytes);

/* Channel bus as a second queued stage (an extension; the paper gives the package 16 host channels of 64 bits,
 * Evaluation setup, but no bus model; the definition is this library's).  After hbf_enable_channel_bus, a read's
 * data-out transfer is no longer a fixed latency after its array time: when the array is done with the read, the
 * transfer queues on the bus of the read's channel, first come first served in (array-done time, index) order
 * behind whatever earlier batches left there, and holds the bus for the transfer time; the read completes when its
 * transfer does.  Programs are unchanged (their transfer stays a latency before the array time), and so are the
 * queue state and the per-die statistics.  The stage runs inside hbf_submit_batch after the array stage (a radix
 * sort of the reads by channel and array-done time, then a segmented max-plus scan); hbf_workspace_bytes grows by
 * 4 bytes per access once it is on.  Array-done times are sort keys of 47 bits here (a restriction of this library, like
 * HBF_ISSUE_LIMIT): a batch whose largest completion time would reach 2^47 ns is refused with HBF_E_INVAL before anything
 * is committed (outputs zeroed, queue, bus and energy state unchanged); the context stays usable.
 * hbf_get_bus_busy_until synchronises and copies the per-channel bus state to host_out [channels]; hbf_reset clears
 * it.  With hbf_submit_batch_paged the stage queues parts (see there); its workspace then holds 4 bytes per part. */
HBF_API int hbf_enable_channel_bus(hbf_ctx *ctx);
HBF_API int hbf_get_bus_busy_until(hbf_ctx *ctx, int64_t *host_out, uint64_t cap);

/* Time-bin power integration (Section "Design", the event-based energy model: a ledger of energy per time bin; a
 * long event is shared among the bins it touches by the time spent in each; P = E / dt + P_idle).  After hbf_enable_energy_bins, hbf_submit_batch books the energy of every
 * modeled access into the bins its array service interval [start, start + s) overlaps, instead of adding the
 * batch's energy to the pending totals: whole pJ, floor(E * overlap / s) per bin, the event's last bin takes
 * what is left.  The ledger is a ring of n_bins bins of bin_ns each, starting at the bin the thermal clock
 * stands in (bin 0 after enable or hbf_reset); time before that bin is booked into it, time past the ring's
 * end into its last bin.  hbf_thermal_step must then be called with dt_ns == bin_ns (HBF_E_INVAL otherwise):
 * it consumes the clock's bin and advances the clock by one.  hbf_get_energy_bins synchronises and copies the
 * ring to host_out [n_bins][channels*dies] (row k = bin *first_bin + k).  The ledger is library-owned device
 * memory allocated by hbf_enable_energy_bins.  With hbf_submit_batch_paged every part is an event (see there). */
HBF_API int hbf_enable_energy_bins(hbf_ctx *ctx, int64_t bin_ns, uint32_t n_bins);
HBF_API int hbf_get_energy_bins(hbf_ctx *ctx, int64_t *host_out, uint64_t cap, int64_t *first_bin);

/* Waits for the last submitted batch and copies its summary to host_out; returns its code. */
HBF_API int hbf_last_result(hbf_ctx *ctx, hbf_batch_result_t *host_out);

/* Advances the package thermal model by dt_ns (Eq. 1, explicit Euler in n_sub substeps): the energy
 * the batches since the last step charged to each die becomes power over this window (P = E/dt +
 * idle, Design D3), ext_power_w (host, [n_regions], nullable with n_ext = 0) adds the external power
 * of each region; then the HBF hotspot drives the four-state throttle controller, whose mode and
 * service fraction the next batch snapshots.  d_temps_out (device [grid_h*grid_w], nullable) receives
 * the field in degrees C.  hot_c_out (host [3], nullable): hottest HBF, HBM and GPU cell; passing it
 * makes the call wait for the step.  Refuses (HBF_E_INVAL) a substep longer than the stability limit. */
HBF_API int hbf_thermal_step(hbf_ctx *ctx, int64_t dt_ns, const float *ext_power_w, uint32_t n_ext,
                     float *d_temps_out, float *hot_c_out);

/* Sets the mode and service fraction directly: the paper's "declared constant" source for
 * deterministic experiments (Design D3). */
HBF_API int hbf_force_mode(hbf_ctx *ctx, int32_t mode, int64_t q_ppm);
HBF_API int hbf_get_mode(hbf_ctx *ctx, int32_t *mode, int64_t *q_ppm);           /* waits for pending work */
HBF_API int hbf_reset(hbf_ctx *ctx);                                             /* queues idle, field at ambient, mode Normal */

/* Chooses how batches are ordered: HBF_PATH_AUTO (default) serves a batch whose records arrive in
 * non-decreasing issue order without a global sort and falls back to the radix sort otherwise (also for a batch in
 * which a single access's service time reaches 2^33 ns, 2^32 ns with retention on: the in-order kernels keep
 * per-tile sums of service times in 56 bits; batches of at most 8,192 records take a route of their own that has no such
 * limit);
 * HBF_PATH_SORT always sorts (a batch already in issue order is sorted on its queue bits only, which a
 * stable sort allows); HBF_PATH_SORT_FULL sorts on every key bit regardless; HBF_PATH_INORDER is the caller's
 * declaration that its batches are in issue order: only the in-order kernels are launched, and a batch that is not in
 * issue order, or has such a long service time (and more than 8,192 records), is refused with HBF_E_INVAL.  All give
 * identical results. */
HBF_API int hbf_set_path(hbf_ctx *ctx, int32_t path);
/* (No step of the method is defined by the next three calls: they steer how the library spreads a batch over the device.)
 * Tile sizes of the in-order path from measurements, on by default: when a batch fills one wave of the device (two tiles
 * per SM), every block of the streaming pass leaves how long its tile took, and later batches size their tiles in
 * proportion to the rates measured at each place (the SMs of a device are not equally fast, and the pass lasts as long as
 * its slowest block).  The record is read through an asynchronous copy that nothing waits for.  Results never depend on
 * where tiles begin; 0 switches the measurements off (tiles in two fixed sizes), which makes run times reproducible from
 * the first batch on.  Waits for nothing. */
HBF_API int hbf_set_tile_balance(hbf_ctx *ctx, int32_t on);
/* The record those sizes come from, as the last batch that filled a wave left it: for each of its tiles (a tile = a place:
 * SM and kind of block) the records it had and the nanoseconds its block took (0: taken out of turn, not measured).
 * Waits for the stream.  *count = number of tiles (0: no such batch yet); with records_out and ns_out (host, [cap]) the values. */
HBF_API int hbf_get_tile_times(hbf_ctx *ctx, uint32_t *records_out, uint32_t *ns_out, uint32_t cap, uint32_t *count);
/* Head entries of the in-order path: how many of the first accesses of every (tile, queue) the streaming pass keeps for the
 * pass that corrects the results of queues that were busy when their tile began.  0 (the default): from measurements, as
 * the tile sizes (the number follows how many queues the last batch that filled a wave left to the slower correction:
 * 3 to 6); 1 to 6: fixed.  Results never depend on it.  HBF_E_INVAL above 6.  Waits for nothing. */
HBF_API int hbf_set_head_entries(hbf_ctx *ctx, uint32_t entries);
/* Thermal step implementation: 0 (default) runs the whole step in one launch of a thread-block cluster when
 * the grid fits its registers and shared memory (up to 32,768 cells with the portable cluster of 8 blocks, 65,536 where
 * the device can place a cluster of 16), else one launch per substep; 1 always uses the latter.
 * Both perform the same arithmetic in the same order (Eq. 1). */
HBF_API int hbf_set_thermal_path(hbf_ctx *ctx, int32_t generic_only);

/* State snapshot (host blob): header, busy_until[queues], pending energy[dies], thermal field and its compensation
 * term; then, for whatever is switched on: the channel buses' busy-until, the energy ledger with its clock, the whole
 * retention state (counters, per-block damage / disturb / cycles / epoch / worn flag, the plan ring).  A blob goes back
 * only into a context with the same geometry and the same things switched on at the same sizes (HBF_E_INVAL otherwise): a
 * long coupled run can be stopped and resumed, or two implementations re-synchronised, at any batch boundary.  Call with
 * host_buf NULL to get the size.  A reduced-order model's state is its own (hbf_rom_get_state). */
HBF_API int hbf_get_state(hbf_ctx *ctx, void *host_buf, size_t *bytes);
HBF_API int hbf_set_state(hbf_ctx *ctx, const void *host_buf, size_t bytes);
/* Individual state arrays, host outputs; each waits for pending work. */
HBF_API int hbf_get_busy_until(hbf_ctx *ctx, int64_t *host_out, uint64_t cap);
HBF_API int hbf_get_pending_energy(hbf_ctx *ctx, int64_t *host_out, uint64_t cap);
HBF_API int hbf_get_temps(hbf_ctx *ctx, float *host_out, uint64_t cap);
HBF_API double hbf_euler_limit_ns(const hbf_ctx *ctx);

/* The order in which the last batch was served when it went through the sort path: batch indices,
 * queue-major, read back from the workspace of that batch into d_order (device [n]); *count (host)
 * receives the number of modeled accesses. */
HBF_API int hbf_queue_order(hbf_ctx *ctx, const void *d_workspace, uint64_t n, uint32_t *d_order, uint64_t *count);

/* Stage timing.  With profiling on, every submit and thermal step records CUDA events between its
 * kernel groups on the context's stream (no synchronisation).  hbf_get_profile waits for the stream
 * and writes the milliseconds of the last batch's stages to ms_out (host, [HBF_PROF_STAGES]):
 * begin, classify, plan+histogram, sort passes, scan+scatter, finish, in-order path, thermal step.
 * A stage that did not run reads 0. */
#define HBF_PROF_STAGES 8
HBF_API int hbf_set_profiling(hbf_ctx *ctx, int on);
HBF_API int hbf_get_profile(hbf_ctx *ctx, float *ms_out, uint32_t cap);
/* Test support, off by default.  The sort path's kernels wait on one another's tiles (decoupled look-back); every such
 * wait polls a bounded number of times and then gives up: the batch's result becomes HBF_E_TIMEOUT, its outputs are zeroed,
 * no state changes, the context is poisoned (later batches return HBF_E_TIMEOUT until hbf_reset).  This call lets a test
 * see that happen without any real stall: poll_limit replaces the bound (0 = the default, 2^24 polls), and tile `tile` of
 * stage 1 (the first radix pass) or 2 (the scan) publishes nothing, so that every tile behind it runs out of polls and
 * returns.  stage 0 = no tile is silenced.  Nothing here makes a kernel wait without a bound. */
HBF_API int hbf_debug_wait_test(hbf_ctx *ctx, uint32_t poll_limit, uint32_t stage, uint32_t tile);
/* Number of kernels this library has launched from the host in the calling process so far (kernels that the device itself
 * launches, the sort path behind HBF_PATH_AUTO's in-order attempt, are not counted). */
HBF_API uint64_t hbf_kernel_launches(void);

/* Explicit-Euler substeps of the package RC network without any allocation.  (The paper has no
 * counterpart: this entry point exists for callers that are not allowed to allocate device memory,
 * for example a serving loop that cannot afford the device-wide synchronisation cudaMalloc may cause,
 * or a plug-in that must work inside the buffers its host application hands it.)
 *
 * It needs no context.  The caller passes every input and output as device pointers:
 * d_cell_C, d_cell_Gx, d_cell_Gy, d_cell_Gsink, d_cell_power_w [grid_h*grid_w] are read only (same
 * meaning and layout as in hbf_config_t; power in watts per cell); d_theta [grid_h*grid_w] is the
 * field as rise above ambient, advanced in place by n_sub substeps of dt_sub_s seconds (same
 * arithmetic as hbf_thermal_step); d_comp [grid_h*grid_w] is the per-cell compensation term that
 * belongs to d_theta (zero for a fresh field, carried from call to call).  Work is enqueued on
 * cuda_stream (a cudaStream_t, NULL = default stream); the call does not wait for it.
 *
 * The second field buffer the update needs lives in an array built into the library: 256 KiB of
 * device memory on every GPU that loads the library, held until the process exits.  Grids of more
 * than HBF_STATIC_MAX_CELLS cells are refused with HBF_E_WORKSPACE.  No cudaMalloc, cudaFree or
 * allocating library routine is called.  The first call on each device looks the array's device
 * address up (with that device current); make that first call before any stream capture begins.
 * All calls on one GPU share the array, which keeps whatever the last call left in it; nothing in
 * it has to be cleared, because every cell is written before it is read.  Two calls whose kernels
 * overlap on the GPU (different streams) race on it: order them.  The stability limit of the
 * explicit step is not checked here; hbf_euler_limit_ns gives it for a context's floorplan. */
#define HBF_STATIC_MAX_CELLS 65536
HBF_API int hbf_euler_substeps_static(const float *d_cell_C, const float *d_cell_Gx, const float *d_cell_Gy,
                                      const float *d_cell_Gsink, const float *d_cell_power_w, float *d_theta,
                                      float *d_comp, uint32_t grid_h, uint32_t grid_w, uint32_t n_sub,
                                      float dt_sub_s, void *cuda_stream);

/* Reduced-order thermal model at run time (Eq. 2): x[k+1] = A x[k] + B p[k] + b, T[k] = C x[k] + D p[k] + d.
 * The paper fits such a model offline (ERA on unit-step responses of the package operator) and steps it instead
 * of the full grid; the fit is not part of this library (the Python package carries one, era.py), the step is.
 * hbf_rom_create copies the matrices (host, row-major, double; b, D, d may be NULL = zero) to the current device;
 * the state starts at zero.  2 * n_states + n_inputs doubles must fit in 40 KiB (HBF_E_INVAL otherwise).
 * hbf_rom_step runs n_steps steps asynchronously on the stream given at create: d_power [n_steps][n_inputs] and
 * d_temps_out [n_steps][n_outputs] are device arrays of doubles owned by the caller.  The state carries over
 * between calls; hbf_rom_reset zeroes it; hbf_rom_get_state synchronises and copies it to host_out [n_states]. */
typedef struct hbf_rom hbf_rom;
HBF_API int hbf_rom_create(uint32_t n_states, uint32_t n_inputs, uint32_t n_outputs, const double *A, const double *B,
                   const double *b, const double *C, const double *D, const double *d, void *cuda_stream, hbf_rom **out);
HBF_API int hbf_rom_destroy(hbf_rom *rom);
HBF_API int hbf_rom_reset(hbf_rom *rom);
HBF_API int hbf_rom_step(hbf_rom *rom, const double *d_power, uint32_t n_steps, double *d_temps_out);
HBF_API int hbf_rom_get_state(hbf_rom *rom, double *host_out, uint64_t cap);

/* The paper's run-time configuration: the thermal step of a context on a reduced-order model instead of the grid.
 * After hbf_attach_rom, hbf_thermal_step(ctx, dt_ns == the dt_ns given here, ...) forms the same power vector as
 * before (window energy / dt + idle + external, one entry per floorplan region = one model input, so the model
 * needs n_inputs == n_regions), advances the model by one step and runs the throttle controller on the hottest
 * output of each medium: output_kind [n_outputs] (host, copied) gives HBF_KIND_HBF / HBF_KIND_HBM / HBF_KIND_GPU
 * per model output.  hot_c_out reports those three maxima; d_temps_out must be NULL (the grid field is not
 * advanced, HBF_E_INVAL otherwise).  The model must have been created on the context's stream; its state is the
 * caller's to reset (hbf_rom_reset).  hbf_attach_rom(ctx, NULL, NULL, 0) goes back to the grid.
 * hbf_get_rom_temps synchronises and copies the last step's outputs to host_out [n_outputs]. */
HBF_API int hbf_attach_rom(hbf_ctx *ctx, hbf_rom *rom, const int32_t *output_kind, int64_t dt_ns);
HBF_API int hbf_get_rom_temps(hbf_ctx *ctx, double *host_out, uint64_t cap);

/* Retention, refresh and wear (Design D4: "Retention, Refresh, and Wear as Injected Latency").
 * From the paper: per-block state (retention damage, read-disturb counter, zone, program/erase cycles used and
 * allowed); lifetime L(T) = L_ref * exp[(E_a/k_B)(1/T - 1/T_ref)] (first equation of D4; E_a = 1.04 eV in the
 * evaluation); damage update D <- D + a_t * dt / L(T) (second equation of D4); eligibility at the lead threshold or
 * at the disturb limit; refresh work of one read + one rewrite per page, sorted by (eligibility epoch; channels in
 * rotation; dies in rotation; zone; block; page); the work is a debt, an admitted access takes over no more than
 * one quantum, whose Eq.-3-scaled service is reserved ahead of its own; a block's cycle count rises and its
 * counters clear once its last quantum is served; debt drained by idle time is accounted separately.
 * What is this library's definition (the paper gives no layout or numbers for it): a block is pages_per_block
 * consecutive pages of one plane, block = (page / pages_per_block) mod blocks_per_plane, id = ((channel * dies +
 * die) * planes + plane) * blocks_per_plane + block, zone = block / blocks_per_zone; a quantum is one page (id =
 * block id * pages_per_block + page), costing t_read + t_prog of array time scaled by Eq. 3 on the CLAIMING
 * access's queue and die, its energy (one page read + one page program) booked on that die; within a die blocks
 * are ordered by (zone, plane, block); a read adds its page count to the disturb counter of the block of its first
 * page, programs add nothing; the modeled accesses of a batch claim in index (ticket) order; commits take effect
 * when the batch, or the decay, that claimed a block's last quantum has completed.
 *
 * hbf_enable_retention: allocates the block state (all fresh).  With hbf_submit_batch_paged the parts claim and disturb (see there).  The
 *   channel-bus stage works on top of it unchanged (claims lengthen the array stage only).  With the energy bins on, a claimed quantum is an event of its
 *   own in the ledger: its energy over the interval in which it was served, ahead of the claiming access's event.
 * hbf_retention_advance: one epoch, asynchronously on the context's stream.  Every block that is not worn out gains
 *   accel * dt / L(T) of damage, T being the temperature of its die's floorplan region: region_temp_c [n_regions]
 *   (host, deg C, copied before the call returns; one entry when the context has no thermal configuration), or
 *   NULL = the hottest cell of each region in the context's thermal field (HBF_E_INVAL without a field, or with a
 *   reduced-order model attached).  Blocks that reach lead_threshold or disturb_limit become eligible in this epoch
 *   and their pages join the end of the plan in the order above.
 * hbf_submit_batch with retention on: the first (planned - claimed - decayed) modeled accesses of the batch, by
 *   index, claim one quantum each; d_die_stats[].busy_ns and the summary's service_ns include the claimed time,
 *   energy_pj does not (it goes to the pending thermal energy).  A refused batch claims nothing and disturbs
 *   nothing.  Every path applies the claims.
 * hbf_retention_decay: idle_ns of idle time drain floor(idle_ns / scaled quantum time) outstanding quanta.
 * hbf_get_retention_blocks / _plan / _totals synchronise the stream and copy to host memory: per-block arrays
 *   [n_blocks] (each nullable); the outstanding quanta in plan order (quanta == NULL: count only); the counters.
 * hbf_reset returns every block to fresh and empties the plan.  The block state and the plan are library-owned
 * device memory (33 bytes per block, 4 bytes per page of the medium). */
typedef struct {
    uint32_t pages_per_block, blocks_per_plane, blocks_per_zone;   /* blocks_per_plane a multiple of blocks_per_zone */
    uint32_t max_pec;                      /* a block that has committed this many cycles is worn out: no more damage, never eligible */
    uint32_t disturb_limit;                /* page reads that make a block eligible; 0 = no limit */
    uint32_t pad;
    double l_ref_s, t_ref_c, ea_ev;        /* lifetime (s) at the reference temperature (deg C); activation energy (eV) */
    double accel;                          /* a_t: reliability-time acceleration */
    double lead_threshold;                 /* damage at which a block becomes eligible */
} hbf_retention_config_t;
typedef struct {
    uint64_t n_blocks, planned, claimed, decayed, commits, worn_blocks, waiting_blocks;
    uint32_t epoch, pad;
} hbf_retention_totals_t;
HBF_API int hbf_enable_retention(hbf_ctx *ctx, const hbf_retention_config_t *cfg);
HBF_API int hbf_retention_advance(hbf_ctx *ctx, int64_t dt_ns, const double *region_temp_c);
HBF_API int hbf_retention_decay(hbf_ctx *ctx, int64_t idle_ns);
HBF_API int hbf_get_retention_blocks(hbf_ctx *ctx, double *damage, uint32_t *disturb, uint32_t *pec, uint32_t *epoch, uint64_t cap);
HBF_API int hbf_get_retention_plan(hbf_ctx *ctx, uint32_t *quanta, uint64_t cap, uint64_t *count);
HBF_API int hbf_get_retention_totals(hbf_ctx *ctx, hbf_retention_totals_t *out);

HBF_API const char *hbf_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif
