/*
 * hbfo.c -- sequential CPU oracle of the HBF service model.  TEST INFRASTRUCTURE ONLY; see hbfo.h.
 *
 * Every step is the plain definition: ranges are found by linear scan, addresses are decoded with
 * '/' and '%', each queue is a list sorted by (issue time, batch index) and served one access at a
 * time, the thermal field is advanced cell by cell in double precision.  No blocking, no fusion.
 */
#include "hbfo.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

typedef struct { uint64_t base, length, media_offset; uint32_t perms, kind, stream_tag, id; } range_t;

struct hbfo_ctx {
    hbfo_config_t cfg;
    uint32_t n_queues, n_dies;
    size_t n_cells;
    range_t ranges[HBFO_MAX_RANGES];
    uint32_t n_ranges, next_range_id;
    int64_t *busy_until;       /* [n_queues] */
    int64_t *pending_pj;       /* [n_dies]   */
    int32_t mode; int64_t q_ppm;
    hbfo_batch_result_t last;
    uint32_t *order; uint64_t order_count, order_cap;
    /* channel bus as a second queued stage (off while bus_busy == NULL) */
    int64_t *bus_busy;         /* [channels] */
    /* time-bin energy ledger (off while bin_ns == 0) */
    int64_t bin_ns; uint32_t n_bins; int64_t cur_bin;
    int64_t *ledger;           /* [n_bins][n_dies], row = bin index modulo n_bins */
    /* thermal */
    int thermal;
    double *C, *Gx, *Gy, *Gs, *T, *Tn, *P;
    int32_t *cell_region, *die_region, *region_kind;
    double *region_idle_w, *region_cells;
    double euler_limit_s;
    struct hbfo_retention *ret;   /* retention, refresh and wear (off while NULL) */
};

/* ---- small helpers ---------------------------------------------------------------------- */

static int is_pow2_u32(uint32_t v) { return v != 0 && (v & (v - 1)) == 0; }

static int64_t ceil_div_i64(int64_t a, int64_t b) { return (a + b - 1) / b; }   /* a >= 0, b > 0 */

static double *dup_f32_as_f64(const float *src, size_t n) {
    double *d = (double *)malloc(n * sizeof(double));
    if (d) for (size_t i = 0; i < n; ++i) d[i] = (double)src[i];
    return d;
}
static int32_t *dup_i32(const int32_t *src, size_t n) {
    int32_t *d = (int32_t *)malloc(n * sizeof(int32_t));
    if (d) memcpy(d, src, n * sizeof(int32_t));
    return d;
}

const char *hbfo_strerror(int code) {
    switch (code) {
    case HBFO_OK: return "ok";
    case HBFO_E_INVAL: return "invalid argument";
    case HBFO_E_RANGE_OVERLAP: return "range overlaps a registered range";
    case HBFO_E_RANGE_FULL: return "range table full";
    case HBFO_E_CAPACITY: return "range exceeds media capacity";
    case HBFO_E_WORKSPACE: return "workspace too small";
    case HBFO_E_CUDA: return "device error";
    case HBFO_E_ACCESS_FAULT: return "batch refused: fail-closed access";
    case HBFO_E_THROTTLED: return "throttled: new reservations withheld";
    case HBFO_E_LINK_SHUTDOWN: return "link shutdown";
    case HBFO_E_TIMEOUT: return "bounded wait expired";
    case HBFO_E_NOMEM: return "out of memory";
    default: return "unknown";
    }
}

/* ---- create / destroy --------------------------------------------------------------------- */

static void free_retention(struct hbfo_retention *r);

static void free_ctx(hbfo_ctx *c) {
    if (!c) return;
    free_retention(c->ret);
    free(c->busy_until); free(c->pending_pj); free(c->order); free(c->ledger); free(c->bus_busy);
    free(c->C); free(c->Gx); free(c->Gy); free(c->Gs); free(c->T); free(c->Tn); free(c->P);
    free(c->cell_region); free(c->die_region); free(c->region_kind);
    free(c->region_idle_w); free(c->region_cells);
    free(c);
}

int hbfo_create(const hbfo_config_t *cfg, hbfo_ctx **out) {
    if (!cfg || !out) return HBFO_E_INVAL;
    if (cfg->channels == 0 || cfg->dies == 0 || cfg->planes == 0) return HBFO_E_INVAL;
    if (!is_pow2_u32(cfg->page_bytes) || !is_pow2_u32(cfg->stripe_bytes)) return HBFO_E_INVAL;
    if (cfg->stripe_bytes < cfg->page_bytes) return HBFO_E_INVAL;
    if (!is_pow2_u32(cfg->read_granule) || !is_pow2_u32(cfg->prog_granule)) return HBFO_E_INVAL;
    if (cfg->queue_level > 1) return HBFO_E_INVAL;
    if (cfg->t_read_ns <= 0 || cfg->t_prog_ns <= 0 || cfg->chan_bytes_per_us == 0) return HBFO_E_INVAL;
    if (cfg->e_cmd_read_pj < 0 || cfg->e_byte_read_pj < 0 || cfg->e_cmd_prog_pj < 0 || cfg->e_byte_prog_pj < 0)
        return HBFO_E_INVAL;
    if (cfg->q_light_ppm < 1 || cfg->q_light_ppm > 1000000) return HBFO_E_INVAL;
    uint64_t nd = (uint64_t)cfg->channels * cfg->dies;
    uint64_t nq = cfg->queue_level == 0 ? nd * cfg->planes : nd;
    if (nq > 65536 || nd > 65536) return HBFO_E_INVAL;

    hbfo_ctx *c = (hbfo_ctx *)calloc(1, sizeof(*c));
    if (!c) return HBFO_E_NOMEM;
    c->cfg = *cfg;
    c->n_queues = (uint32_t)nq; c->n_dies = (uint32_t)nd;
    c->busy_until = (int64_t *)calloc(nq, sizeof(int64_t));
    c->pending_pj = (int64_t *)calloc(nd, sizeof(int64_t));
    if (!c->busy_until || !c->pending_pj) { free_ctx(c); return HBFO_E_NOMEM; }
    c->mode = HBFO_MODE_NORMAL; c->q_ppm = 1000000;

    c->thermal = cfg->cell_C != NULL;
    if (c->thermal) {
        if (cfg->grid_h == 0 || cfg->grid_w == 0 || cfg->n_sub == 0 || cfg->n_regions == 0 ||
            !cfg->cell_Gx || !cfg->cell_Gy || !cfg->cell_Gsink || !cfg->cell_region || !cfg->die_region ||
            !cfg->region_kind || !cfg->region_idle_w) { free_ctx(c); return HBFO_E_INVAL; }
        if (!(cfg->rtt_c < cfg->ltt_c && cfg->ltt_c < cfg->stt_c && cfg->stt_c < cfg->shutdown_c)) {
            free_ctx(c); return HBFO_E_INVAL;
        }
        size_t nc = (size_t)cfg->grid_h * cfg->grid_w;
        c->n_cells = nc;
        c->C = dup_f32_as_f64(cfg->cell_C, nc);  c->Gx = dup_f32_as_f64(cfg->cell_Gx, nc);
        c->Gy = dup_f32_as_f64(cfg->cell_Gy, nc); c->Gs = dup_f32_as_f64(cfg->cell_Gsink, nc);
        c->T = (double *)malloc(nc * sizeof(double)); c->Tn = (double *)malloc(nc * sizeof(double));
        c->P = (double *)calloc(nc, sizeof(double));
        c->cell_region = dup_i32(cfg->cell_region, nc);
        c->die_region = dup_i32(cfg->die_region, nd);
        c->region_kind = dup_i32(cfg->region_kind, cfg->n_regions);
        c->region_idle_w = dup_f32_as_f64(cfg->region_idle_w, cfg->n_regions);
        c->region_cells = (double *)calloc(cfg->n_regions, sizeof(double));
        if (!c->C || !c->Gx || !c->Gy || !c->Gs || !c->T || !c->Tn || !c->P || !c->cell_region ||
            !c->die_region || !c->region_kind || !c->region_idle_w || !c->region_cells) {
            free_ctx(c); return HBFO_E_NOMEM;
        }
        for (size_t i = 0; i < nc; ++i) {
            if (!(c->C[i] > 0.0) || c->Gx[i] < 0.0 || c->Gy[i] < 0.0 || c->Gs[i] < 0.0) { free_ctx(c); return HBFO_E_INVAL; }
            int32_t g = c->cell_region[i];
            if (g >= (int32_t)cfg->n_regions) { free_ctx(c); return HBFO_E_INVAL; }
            if (g >= 0) c->region_cells[g] += 1.0;
            c->T[i] = (double)cfg->ambient_c;          /* the field starts at ambient everywhere */
        }
        for (uint64_t d = 0; d < nd; ++d) {
            int32_t g = c->die_region[d];
            if (g < 0 || g >= (int32_t)cfg->n_regions || c->region_cells[g] == 0.0) { free_ctx(c); return HBFO_E_INVAL; }
        }
        /* largest stable explicit step: min over cells of C / (sum of conductances on the cell) */
        uint32_t H = cfg->grid_h, W = cfg->grid_w;
        double lim = INFINITY;
        for (uint32_t y = 0; y < H; ++y) for (uint32_t x = 0; x < W; ++x) {
            size_t i = (size_t)y * W + x;
            double g = c->Gs[i];
            if (x + 1 < W) g += c->Gx[i];
            if (x > 0)     g += c->Gx[i - 1];
            if (y + 1 < H) g += c->Gy[i];
            if (y > 0)     g += c->Gy[i - W];
            if (g > 0.0 && c->C[i] / g < lim) lim = c->C[i] / g;
        }
        c->euler_limit_s = lim;
    }
    *out = c;
    return HBFO_OK;
}

int hbfo_destroy(hbfo_ctx *ctx) { free_ctx(ctx); return HBFO_OK; }

double hbfo_euler_limit_ns(hbfo_ctx *ctx) { return ctx && ctx->thermal ? ctx->euler_limit_s * 1e9 : 0.0; }

static void retention_reset(struct hbfo_retention *r);

int hbfo_reset(hbfo_ctx *c) {
    if (!c) return HBFO_E_INVAL;
    memset(c->busy_until, 0, c->n_queues * sizeof(int64_t));
    memset(c->pending_pj, 0, c->n_dies * sizeof(int64_t));
    c->mode = HBFO_MODE_NORMAL; c->q_ppm = 1000000;
    memset(&c->last, 0, sizeof(c->last));
    c->order_count = 0;
    c->cur_bin = 0;
    if (c->bus_busy) memset(c->bus_busy, 0, c->cfg.channels * sizeof(int64_t));
    if (c->ledger) memset(c->ledger, 0, (size_t)c->n_bins * c->n_dies * sizeof(int64_t));
    if (c->thermal) for (size_t i = 0; i < c->n_cells; ++i) c->T[i] = (double)c->cfg.ambient_c;
    retention_reset(c->ret);
    return HBFO_OK;
}

int hbfo_force_mode(hbfo_ctx *c, int32_t mode, int64_t q_ppm) {
    if (!c || mode < 0 || mode > 3 || q_ppm < 1 || q_ppm > 1000000) return HBFO_E_INVAL;
    c->mode = mode; c->q_ppm = q_ppm;
    return HBFO_OK;
}

int hbfo_get_mode(hbfo_ctx *c, int32_t *mode, int64_t *q_ppm) {
    if (!c) return HBFO_E_INVAL;
    if (mode) *mode = c->mode;
    if (q_ppm) *q_ppm = c->q_ppm;
    return HBFO_OK;
}

/* ---- ranges (Design D1) -------------------------------------------------------------------- */

int hbfo_register_range(hbfo_ctx *c, uint64_t base, uint64_t length, uint32_t perms, uint32_t kind,
                        uint32_t stream_tag, uint64_t media_offset, uint32_t *out_id) {
    if (!c || length == 0 || (perms & ~3u) || perms == 0 || kind > 1) return HBFO_E_INVAL;
    if (base + length < base) return HBFO_E_INVAL;                       /* wraps the address space */
    if (media_offset + length < media_offset) return HBFO_E_INVAL;
    if (c->cfg.capacity_bytes && media_offset + length > c->cfg.capacity_bytes) return HBFO_E_CAPACITY;
    if (c->n_ranges == HBFO_MAX_RANGES) return HBFO_E_RANGE_FULL;
    for (uint32_t g = 0; g < c->n_ranges; ++g) {
        const range_t *r = &c->ranges[g];
        if (base < r->base + r->length && r->base < base + length) return HBFO_E_RANGE_OVERLAP;
    }
    range_t *r = &c->ranges[c->n_ranges++];
    r->base = base; r->length = length; r->media_offset = media_offset;
    r->perms = perms; r->kind = kind; r->stream_tag = stream_tag; r->id = c->next_range_id++;
    if (out_id) *out_id = r->id;
    return HBFO_OK;
}

int hbfo_clear_ranges(hbfo_ctx *c) { if (!c) return HBFO_E_INVAL; c->n_ranges = 0; return HBFO_OK; }

/* Classification of one access.  Outside every range: native path.  Inside a range: modeled only
 * if the whole byte span lies in that one range and the operation is permitted; otherwise it fails. */
int hbfo_classify(hbfo_ctx *c, const hbfo_access_t *a, int32_t *range_id) {
    if (range_id) *range_id = -1;
    if (a->bytes == 0 || (a->flags & ~1u) || a->issue_ns < 0)              /* any issue time >= 0 is in the domain */
        return HBFO_ST_UNSUPPORTED;
    for (uint32_t g = 0; g < c->n_ranges; ++g) {                         /* linear scan, on purpose */
        const range_t *r = &c->ranges[g];
        if (a->addr >= r->base && a->addr - r->base < r->length) {
            uint64_t rel = a->addr - r->base;
            if (range_id) *range_id = (int32_t)g;
            if ((uint64_t)a->bytes > r->length - rel) return HBFO_ST_FAULT_PARTIAL;   /* leaves the range (or wraps) */
            uint32_t need = (a->flags & 1u) ? 2u : 1u;                   /* bit0 read, bit1 program */
            if (!(r->perms & need)) return HBFO_ST_FAULT_PERM;
            return HBFO_ST_READY;
        }
    }
    return HBFO_ST_NATIVE;
}

/* ---- decode and service terms --------------------------------------------------------------- */

int hbfo_decode(hbfo_ctx *c, uint64_t off, uint32_t bytes, uint32_t *channel, uint32_t *die,
                uint32_t *plane, uint64_t *row, uint64_t *page, uint64_t *npages, uint32_t *queue) {
    if (!c) return HBFO_E_INVAL;
    const uint64_t Cn = c->cfg.channels, Dn = c->cfg.dies, Pn = c->cfg.planes;
    const uint64_t stripe = c->cfg.stripe_bytes, pg = c->cfg.page_bytes;
    uint64_t u  = off / stripe;                     /* stripe unit: channel first, then die, then plane */
    uint64_t ch = u % Cn;
    uint64_t di = (u / Cn) % Dn;
    uint64_t pl = (u / (Cn * Dn)) % Pn;
    uint64_t rw = u / (Cn * Dn * Pn);
    uint64_t pa = rw * (stripe / pg) + (off % stripe) / pg;
    uint64_t np = ((off % pg) + (uint64_t)bytes + pg - 1) / pg;
    uint64_t q  = c->cfg.queue_level == 0 ? (ch * Dn + di) * Pn + pl : ch * Dn + di;
    if (channel) *channel = (uint32_t)ch;
    if (die) *die = (uint32_t)di;
    if (plane) *plane = (uint32_t)pl;
    if (row) *row = rw;
    if (page) *page = pa;
    if (npages) *npages = np;
    if (queue) *queue = (uint32_t)q;
    return HBFO_OK;
}

int hbfo_service_terms(hbfo_ctx *c, uint32_t bytes, uint64_t npages, uint32_t op, int64_t q_ppm,
                       int64_t *charged_bytes, int64_t *xfer_ns, int64_t *s_ns, int64_t *energy_pj) {
    if (!c || q_ppm < 1 || op > 1) return HBFO_E_INVAL;
    int64_t gran = op ? (int64_t)c->cfg.prog_granule : (int64_t)c->cfg.read_granule;
    int64_t cb   = ceil_div_i64((int64_t)bytes, gran) * gran;           /* bytes charged: whole granules */
    int64_t xfer = ceil_div_i64(cb * 1000, (int64_t)c->cfg.chan_bytes_per_us);
    int64_t s0   = (int64_t)npages * (op ? c->cfg.t_prog_ns : c->cfg.t_read_ns);
    int64_t s    = ceil_div_i64(s0 * 1000000, q_ppm);                   /* Eq. 3 */
    int64_t e    = op ? c->cfg.e_cmd_prog_pj + c->cfg.e_byte_prog_pj * cb
                      : c->cfg.e_cmd_read_pj + c->cfg.e_byte_read_pj * cb;
    if (charged_bytes) *charged_bytes = cb;
    if (xfer_ns) *xfer_ns = xfer;
    if (s_ns) *s_ns = s;
    if (energy_pj) *energy_pj = e;
    return HBFO_OK;
}

/* ---- time-bin power integration (Section "Design", the paragraph on the event-based energy model) -------
 * The ledger holds energy per (bin of bin_ns, die); an event longer than one bin gives each bin it touches the
 * fraction of its energy that matches the time it spent there.  The event of an access is its array service interval
 * [start, start + s) on its die.  Shares are whole pJ: floor(E * overlap / s) for every bin but the event's
 * last, which takes what is left, so a die's bins always add up to its events' energy.  The ledger is a ring
 * of n_bins bins starting at the bin the thermal clock stands in: time before it counts into that bin, time
 * past the ring's end into the ring's last bin. */
int hbfo_enable_energy_bins(hbfo_ctx *c, int64_t bin_ns, uint32_t n_bins) {
    if (!c || bin_ns <= 0 || n_bins == 0) return HBFO_E_INVAL;
    int64_t *l = (int64_t *)calloc((size_t)n_bins * c->n_dies, sizeof(int64_t));
    if (!l) return HBFO_E_NOMEM;
    free(c->ledger);
    c->ledger = l; c->bin_ns = bin_ns; c->n_bins = n_bins; c->cur_bin = 0;
    memset(c->pending_pj, 0, c->n_dies * sizeof(int64_t));
    return HBFO_OK;
}

int hbfo_get_energy_bins(hbfo_ctx *c, int64_t *out, uint64_t cap, int64_t *first_bin) {
    if (!c || !c->ledger || !out || cap < (uint64_t)c->n_bins * c->n_dies) return HBFO_E_INVAL;
    for (uint32_t k = 0; k < c->n_bins; ++k) {              /* row k of the output is bin cur_bin + k */
        int64_t b = c->cur_bin + k;
        memcpy(out + (size_t)k * c->n_dies, c->ledger + (size_t)(b % c->n_bins) * c->n_dies, c->n_dies * sizeof(int64_t));
    }
    if (first_bin) *first_bin = c->cur_bin;
    return HBFO_OK;
}

static void ledger_add(hbfo_ctx *c, uint32_t die, int64_t bin, int64_t pj) {
    if (bin < c->cur_bin) bin = c->cur_bin;
    if (bin > c->cur_bin + (int64_t)c->n_bins - 1) bin = c->cur_bin + (int64_t)c->n_bins - 1;
    c->ledger[(size_t)(bin % c->n_bins) * c->n_dies + die] += pj;
}

static void ledger_event(hbfo_ctx *c, uint32_t die, int64_t start, int64_t s, int64_t energy_pj) {
    const int64_t end = start + s, w = c->bin_ns;             /* s >= 1 */
    const int64_t b0 = start / w, b1 = (end - 1) / w;
    int64_t given = 0;
    for (int64_t b = b0; b < b1; ++b) {
        int64_t lo = b * w > start ? b * w : start, hi = (b + 1) * w;
        int64_t share = (int64_t)(((__int128)energy_pj * (hi - lo)) / s);
        ledger_add(c, die, b, share);
        given += share;
    }
    ledger_add(c, die, b1, energy_pj - given);
}

/* ---- channel bus as a second queued stage (this build's extension; the paper gives the package 16 host channels
 * of 64 bits, Evaluation setup, and a flash back end, but no bus model) ---------------------------------------
 * With the stage on, a read's data-out transfer is no longer a pure latency after its array time: when the array
 * is done with the read (time D), the transfer queues on the bus of the read's channel, first come first served in
 * (D, batch index) order behind whatever earlier batches left on that bus, and occupies it for the transfer time.
 * The read completes when its transfer does.  Programs keep their transfer as a latency before the array time. */
int hbfo_enable_channel_bus(hbfo_ctx *c) {
    if (!c) return HBFO_E_INVAL;
    if (!c->bus_busy) c->bus_busy = (int64_t *)calloc(c->cfg.channels, sizeof(int64_t));
    return c->bus_busy ? HBFO_OK : HBFO_E_NOMEM;
}

int hbfo_get_bus_busy_until(hbfo_ctx *c, int64_t *out, uint64_t cap) {
    if (!c || !c->bus_busy || !out || cap < c->cfg.channels) return HBFO_E_INVAL;
    memcpy(out, c->bus_busy, c->cfg.channels * sizeof(int64_t));
    return HBFO_OK;
}

typedef struct { int64_t done_ns; uint32_t idx; } bent_t;

static int cmp_bent(const void *pa, const void *pb) {
    const bent_t *a = (const bent_t *)pa, *b = (const bent_t *)pb;
    if (a->done_ns != b->done_ns) return a->done_ns < b->done_ns ? -1 : 1;
    if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
    return 0;
}

/* ---- retention, refresh and wear (Design D4) --------------------------------------------------------
 * From the paper (Design D4): per-block state = accumulated retention damage, read-disturb counter, zone,
 * program/erase cycles used and allowed.  Lifetime at temperature T (first equation of D4, Arrhenius form around a
 * reference point; E_a = 1.04 eV in the evaluation): L(T) = L_ref * exp[(E_a / k_B) * (1/T - 1/T_ref)].  Damage
 * update over dt (second equation of D4): D <- D + a_t * dt / L(T).  Eligibility: damage at the lead threshold, or
 * disturb count at its limit.  Refresh work = one read + one rewrite per page, issued sorted by (epoch in which the
 * block became eligible; channels in rotation; dies of a channel in rotation; zone; block; page).  That work is a
 * debt: an admitted access takes over no more than one quantum and has the quantum's service (with Eq. 3 scaling)
 * reserved ahead of its own.  A block's cycle count goes up, and its damage and disturb counters go back to zero,
 * once its last quantum has been served; debt drained by idle time is accounted separately from claimed debt.
 * What is a reading (the paper gives no numbers or layouts for these): a block is pages_per_block consecutive
 * pages of one plane, block = (page / pages_per_block) mod blocks_per_plane, zone = block / blocks_per_zone; a
 * read adds its page count to the disturb counter of the block of its first page, programs add nothing; damage
 * and eligibility are evaluated by hbfo_retention_advance, once per call (= one epoch), with one temperature per
 * floorplan region (given, or the hottest cell of the region in the field); within a die, blocks are ordered by
 * (zone, plane, block); a quantum is one page, read and rewritten: t_read + t_prog of array time, scaled like any
 * service (Eq. 3), charged on the claiming access's own queue and die, its energy booked on that die; the modeled
 * accesses of a batch claim in index (ticket) order; commits take effect when the batch (or the decay) that
 * claimed a block's last quantum has completed; idle time drains one quantum per scaled quantum time. */
#define HBFO_KB_EV 8.617333262e-5                  /* Boltzmann constant, eV/K */

struct hbfo_retention {
    hbfo_retention_config_t cfg;
    uint64_t n_blocks;
    double *damage; uint32_t *disturb, *pec, *epoch_of; uint8_t *worn;
    uint64_t *last_pos;          /* plan position of the block's last quantum */
    uint32_t *plan; uint64_t plan_len, plan_cap;
    uint64_t claimed, decayed, commits, worn_blocks;
    uint32_t epoch;
};

static void free_retention(struct hbfo_retention *r) {
    if (!r) return;
    free(r->damage); free(r->disturb); free(r->pec); free(r->epoch_of); free(r->worn); free(r->last_pos); free(r->plan);
    free(r);
}

static void retention_reset(struct hbfo_retention *r) {
    if (!r) return;
    memset(r->damage, 0, r->n_blocks * sizeof(double)); memset(r->disturb, 0, r->n_blocks * 4);
    memset(r->pec, 0, r->n_blocks * 4); memset(r->epoch_of, 0, r->n_blocks * 4); memset(r->worn, 0, r->n_blocks);
    r->plan_len = 0; r->claimed = r->decayed = r->commits = r->worn_blocks = 0; r->epoch = 0;
}

int hbfo_enable_retention(hbfo_ctx *c, const hbfo_retention_config_t *cfg) {
    if (!c || !cfg || c->ret) return HBFO_E_INVAL;
    if (cfg->pages_per_block == 0 || cfg->blocks_per_plane == 0 || cfg->blocks_per_zone == 0 ||
        cfg->blocks_per_plane % cfg->blocks_per_zone != 0 || cfg->max_pec == 0) return HBFO_E_INVAL;
    if (!(cfg->l_ref_s > 0.0) || !(cfg->t_ref_c > -273.15) || !(cfg->ea_ev >= 0.0) || !(cfg->accel > 0.0) ||
        !(cfg->lead_threshold > 0.0)) return HBFO_E_INVAL;
    const uint64_t nb = (uint64_t)c->cfg.channels * c->cfg.dies * c->cfg.planes * cfg->blocks_per_plane;
    if (nb * cfg->pages_per_block > 0xffffffffull) return HBFO_E_INVAL;
    struct hbfo_retention *r = (struct hbfo_retention *)calloc(1, sizeof(*r));
    if (!r) return HBFO_E_NOMEM;
    r->cfg = *cfg; r->n_blocks = nb;
    r->damage = (double *)calloc(nb, sizeof(double)); r->disturb = (uint32_t *)calloc(nb, 4);
    r->pec = (uint32_t *)calloc(nb, 4); r->epoch_of = (uint32_t *)calloc(nb, 4); r->worn = (uint8_t *)calloc(nb, 1);
    r->last_pos = (uint64_t *)calloc(nb, 8);
    if (!r->damage || !r->disturb || !r->pec || !r->epoch_of || !r->worn || !r->last_pos) { free_retention(r); return HBFO_E_NOMEM; }
    c->ret = r;
    return HBFO_OK;
}

double hbfo_retention_lifetime_s(hbfo_ctx *c, double temp_c) {
    if (!c || !c->ret) return 0.0;
    const hbfo_retention_config_t *k = &c->ret->cfg;
    const double T = temp_c + 273.15, Tref = k->t_ref_c + 273.15;
    return k->l_ref_s * exp((k->ea_ev / HBFO_KB_EV) * (1.0 / T - 1.0 / Tref));
}

/* the block an access's first page lies in: ((channel, die, plane) * blocks_per_plane + block) */
static uint64_t retention_block_of(hbfo_ctx *c, uint64_t off) {
    uint32_t ch, di, pl; uint64_t page;
    hbfo_decode(c, off, 1, &ch, &di, &pl, NULL, &page, NULL, NULL);
    const struct hbfo_retention *r = c->ret;
    const uint64_t bip = (page / r->cfg.pages_per_block) % r->cfg.blocks_per_plane;
    return (((uint64_t)ch * c->cfg.dies + di) * c->cfg.planes + pl) * r->cfg.blocks_per_plane + bip;
}

/* blocks whose last quantum lies below the watermark commit: one cycle, counters cleared */
static void retention_commit(struct hbfo_retention *r) {
    const uint64_t mark = r->claimed + r->decayed;
    for (uint64_t b = 0; b < r->n_blocks; ++b) {
        if (r->epoch_of[b] == 0 || r->last_pos[b] >= mark) continue;
        r->pec[b] += 1; r->damage[b] = 0.0; r->disturb[b] = 0; r->epoch_of[b] = 0; r->commits += 1;
        if (r->pec[b] >= r->cfg.max_pec) { r->worn[b] = 1; r->worn_blocks += 1; }
    }
}

static int retention_plan_push(struct hbfo_retention *r, uint32_t quantum) {
    if (r->plan_len == r->plan_cap) {
        uint64_t cap = r->plan_cap ? r->plan_cap * 2 : 1024;
        uint32_t *p = (uint32_t *)realloc(r->plan, cap * 4);
        if (!p) return HBFO_E_NOMEM;
        r->plan = p; r->plan_cap = cap;
    }
    r->plan[r->plan_len++] = quantum;
    return HBFO_OK;
}

int hbfo_retention_advance(hbfo_ctx *c, int64_t dt_ns, const double *region_temp_c) {
    if (!c || !c->ret || dt_ns < 0) return HBFO_E_INVAL;
    struct hbfo_retention *r = c->ret;
    const uint32_t NR = c->thermal ? c->cfg.n_regions : 1;
    if (!region_temp_c && !c->thermal) return HBFO_E_INVAL;
    double *temp = (double *)malloc(NR * sizeof(double));
    if (!temp) return HBFO_E_NOMEM;
    if (region_temp_c) memcpy(temp, region_temp_c, NR * sizeof(double));
    else {                                                     /* the hottest cell of each region */
        for (uint32_t k = 0; k < NR; ++k) temp[k] = -INFINITY;
        for (size_t i = 0; i < c->n_cells; ++i) {
            int32_t g = c->cell_region[i];
            if (g >= 0 && c->T[i] > temp[g]) temp[g] = c->T[i];
        }
        for (uint32_t k = 0; k < NR; ++k) if (temp[k] == -INFINITY) temp[k] = (double)c->cfg.ambient_c;
    }
    r->epoch += 1;
    const uint32_t Cn = c->cfg.channels, Dn = c->cfg.dies, Pn = c->cfg.planes;
    const uint32_t bpp = r->cfg.blocks_per_plane, bpz = r->cfg.blocks_per_zone, ppb = r->cfg.pages_per_block;
    const double dt_s = (double)dt_ns * 1e-9;
    /* damage, then eligibility */
    for (uint64_t b = 0; b < r->n_blocks; ++b) {
        if (r->worn[b]) continue;
        const uint64_t die = b / ((uint64_t)Pn * bpp);
        const uint32_t g = c->thermal ? (uint32_t)c->die_region[die] : 0u;
        r->damage[b] += r->cfg.accel * dt_s / hbfo_retention_lifetime_s(c, temp[g]);
        if (r->epoch_of[b] == 0 && (r->damage[b] >= r->cfg.lead_threshold ||
                                    (r->cfg.disturb_limit && r->disturb[b] >= r->cfg.disturb_limit)))
            r->epoch_of[b] = r->epoch;
    }
    free(temp);
    /* this epoch's quanta: per die in (zone, plane, block, page) order ... */
    const uint32_t n_dies = Cn * Dn;
    uint32_t **list = (uint32_t **)calloc(n_dies, sizeof(uint32_t *));
    uint64_t *len = (uint64_t *)calloc(n_dies, 8), *pos = (uint64_t *)calloc(n_dies, 8);
    uint32_t *die_ptr = (uint32_t *)calloc(Cn, 4);
    int rc = HBFO_OK;
    uint64_t remaining = 0;
    if (!list || !len || !pos || !die_ptr) { rc = HBFO_E_NOMEM; goto done; }
    for (uint32_t d = 0; d < n_dies; ++d) {
        uint64_t cnt = 0;
        for (uint32_t pl = 0; pl < Pn; ++pl)
            for (uint32_t k = 0; k < bpp; ++k)
                if (r->epoch_of[((uint64_t)d * Pn + pl) * bpp + k] == r->epoch) ++cnt;
        if (!cnt) continue;
        list[d] = (uint32_t *)malloc(cnt * ppb * 4);
        if (!list[d]) { rc = HBFO_E_NOMEM; goto done; }
        for (uint32_t z = 0; z < bpp / bpz; ++z)
            for (uint32_t pl = 0; pl < Pn; ++pl)
                for (uint32_t k = z * bpz; k < (z + 1) * bpz; ++k) {
                    const uint64_t b = ((uint64_t)d * Pn + pl) * bpp + k;
                    if (r->epoch_of[b] != r->epoch) continue;
                    for (uint32_t pg = 0; pg < ppb; ++pg) list[d][len[d]++] = (uint32_t)(b * ppb + pg);
                }
        remaining += len[d];
    }
    /* ... emitted one at a time: channels in turn, within a channel its dies in turn, skipping what is exhausted */
    for (uint32_t ch = 0; remaining; ch = (ch + 1) % Cn) {
        int left = 0;
        for (uint32_t di = 0; di < Dn; ++di) if (pos[ch * Dn + di] < len[ch * Dn + di]) left = 1;
        if (!left) continue;
        uint32_t di = die_ptr[ch];
        while (pos[ch * Dn + di] >= len[ch * Dn + di]) di = (di + 1) % Dn;
        const uint32_t d = ch * Dn + di;
        const uint32_t quantum = list[d][pos[d]++];
        r->last_pos[quantum / ppb] = r->plan_len;            /* pages go out in order: the last one stays */
        rc = retention_plan_push(r, quantum);
        if (rc != HBFO_OK) goto done;
        die_ptr[ch] = (di + 1) % Dn;
        --remaining;
    }
done:
    if (list) for (uint32_t d = 0; d < n_dies; ++d) free(list[d]);
    free(list); free(len); free(pos); free(die_ptr);
    return rc;
}

/* scaled array time of one quantum: a page read and a page program (Eq. 3) */
static int64_t retention_quantum_ns(hbfo_ctx *c, int64_t q_ppm) {
    return ceil_div_i64((c->cfg.t_read_ns + c->cfg.t_prog_ns) * 1000000, q_ppm);
}
static int64_t retention_quantum_pj(hbfo_ctx *c) {
    const int64_t pg = (int64_t)c->cfg.page_bytes;
    return c->cfg.e_cmd_read_pj + c->cfg.e_byte_read_pj * pg + c->cfg.e_cmd_prog_pj + c->cfg.e_byte_prog_pj * pg;
}

int hbfo_retention_decay(hbfo_ctx *c, int64_t idle_ns) {
    if (!c || !c->ret || idle_ns < 0) return HBFO_E_INVAL;
    struct hbfo_retention *r = c->ret;
    uint64_t drained = (uint64_t)(idle_ns / retention_quantum_ns(c, c->q_ppm));
    const uint64_t debt = r->plan_len - (r->claimed + r->decayed);
    if (drained > debt) drained = debt;
    r->decayed += drained;
    retention_commit(r);
    return HBFO_OK;
}

int hbfo_get_retention_blocks(hbfo_ctx *c, double *damage, uint32_t *disturb, uint32_t *pec, uint32_t *epoch, uint64_t cap) {
    if (!c || !c->ret || cap < c->ret->n_blocks) return HBFO_E_INVAL;
    const struct hbfo_retention *r = c->ret;
    if (damage) memcpy(damage, r->damage, r->n_blocks * 8);
    if (disturb) memcpy(disturb, r->disturb, r->n_blocks * 4);
    if (pec) memcpy(pec, r->pec, r->n_blocks * 4);
    if (epoch) memcpy(epoch, r->epoch_of, r->n_blocks * 4);
    return HBFO_OK;
}

int hbfo_get_retention_plan(hbfo_ctx *c, uint32_t *quanta, uint64_t cap, uint64_t *count) {
    if (!c || !c->ret || !count) return HBFO_E_INVAL;
    const struct hbfo_retention *r = c->ret;
    const uint64_t mark = r->claimed + r->decayed, m = r->plan_len - mark;
    *count = m;
    if (!quanta) return HBFO_OK;
    if (cap < m) return HBFO_E_INVAL;
    memcpy(quanta, r->plan + mark, m * 4);
    return HBFO_OK;
}

int hbfo_get_retention_totals(hbfo_ctx *c, hbfo_retention_totals_t *out) {
    if (!c || !c->ret || !out) return HBFO_E_INVAL;
    const struct hbfo_retention *r = c->ret;
    out->planned = r->plan_len; out->claimed = r->claimed; out->decayed = r->decayed; out->commits = r->commits;
    out->worn_blocks = r->worn_blocks; out->epoch = r->epoch; out->n_blocks = r->n_blocks;
    out->waiting_blocks = 0;
    for (uint64_t b = 0; b < r->n_blocks; ++b) if (r->epoch_of[b]) out->waiting_blocks += 1;
    return HBFO_OK;
}

/* ---- submit --------------------------------------------------------------------------------- */

typedef struct { int64_t issue_ns; uint32_t idx; } qent_t;

static int cmp_qent(const void *pa, const void *pb) {
    const qent_t *a = (const qent_t *)pa, *b = (const qent_t *)pb;
    if (a->issue_ns != b->issue_ns) return a->issue_ns < b->issue_ns ? -1 : 1;
    if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
    return 0;
}

int hbfo_submit_batch(hbfo_ctx *c, const hbfo_access_t *acc, uint64_t n, int64_t *completion_ns,
                      int64_t *stall_ns, uint8_t *status, hbfo_die_stats_t *die_stats) {
    if (!c || (n && (!acc || !completion_ns || !stall_ns)) || n > 0xffffffffull) return HBFO_E_INVAL;
    hbfo_batch_result_t res; memset(&res, 0, sizeof(res));
    const int64_t q = c->q_ppm;                               /* snapshot before any reservation */
    res.mode = c->mode; res.q_ppm = q;
    if (c->mode == HBFO_MODE_SHUTDOWN) { res.code = HBFO_E_LINK_SHUTDOWN; c->last = res; return res.code; }
    if (c->mode == HBFO_MODE_SEVERE)   { res.code = HBFO_E_THROTTLED;     c->last = res; return res.code; }

    uint8_t *st = (uint8_t *)malloc(n ? n : 1);
    int32_t *rg = (int32_t *)malloc((n ? n : 1) * sizeof(int32_t));
    if (!st || !rg) { free(st); free(rg); return HBFO_E_NOMEM; }

    /* validate pass: nothing changes if any access fails */
    uint64_t n_fault = 0, n_native = 0, n_ready = 0;
    for (uint64_t i = 0; i < n; ++i) {
        st[i] = (uint8_t)hbfo_classify(c, &acc[i], &rg[i]);
        if (st[i] == HBFO_ST_NATIVE) ++n_native; else if (st[i] == HBFO_ST_READY) ++n_ready; else ++n_fault;
    }
    if (status) memcpy(status, st, n);
    if (die_stats) memset(die_stats, 0, c->n_dies * sizeof(hbfo_die_stats_t));
    if (n_fault) {
        memset(completion_ns, 0, n * sizeof(int64_t)); memset(stall_ns, 0, n * sizeof(int64_t));
        res.code = HBFO_E_ACCESS_FAULT; res.n_fault = n_fault; res.n_native = n_native;
        c->last = res; free(st); free(rg);
        return res.code;
    }

    /* decode + terms */
    uint32_t *queue = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    uint32_t *die   = (uint32_t *)malloc((n ? n : 1) * sizeof(uint32_t));
    int64_t *a_ns = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    int64_t *s_ns = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    int64_t *post = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    int64_t *cbs  = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    int64_t *eng  = (int64_t *)malloc((n ? n : 1) * sizeof(int64_t));
    uint64_t *cnt = (uint64_t *)calloc((size_t)c->n_queues + 1, sizeof(uint64_t));
    qent_t *ent = (qent_t *)malloc((n_ready ? n_ready : 1) * sizeof(qent_t));
    int rc = HBFO_OK;
    uint64_t claims = 0;                                      /* refresh quanta claimed by this batch */
    uint8_t *claimed = (uint8_t *)calloc(n ? n : 1, 1);
    if (!claimed) { rc = HBFO_E_NOMEM; goto done; }
    if (!queue || !die || !a_ns || !s_ns || !post || !cbs || !eng || !cnt || !ent) { rc = HBFO_E_NOMEM; goto done; }
    if (c->order_cap < n_ready) {
        free(c->order); c->order = (uint32_t *)malloc((n_ready ? n_ready : 1) * sizeof(uint32_t));
        if (!c->order) { c->order_cap = 0; rc = HBFO_E_NOMEM; goto done; }
        c->order_cap = n_ready;
    }

    for (uint64_t i = 0; i < n; ++i) {
        if (st[i] != HBFO_ST_READY) continue;
        const range_t *r = &c->ranges[rg[i]];
        uint64_t off = r->media_offset + (acc[i].addr - r->base);
        uint32_t ch, di, pl, qu; uint64_t np;
        hbfo_decode(c, off, acc[i].bytes, &ch, &di, &pl, NULL, NULL, &np, &qu);
        uint32_t op = acc[i].flags & 1u;
        int64_t cb, xfer, s, e;
        hbfo_service_terms(c, acc[i].bytes, np, op, q, &cb, &xfer, &s, &e);
        queue[i] = qu; die[i] = ch * c->cfg.dies + di;
        if (c->ret && c->ret->claimed + c->ret->decayed + claims < c->ret->plan_len) {
            /* this admission claims one refresh quantum: its scaled service is reserved before the access's own */
            s += retention_quantum_ns(c, q);
            if (!c->bin_ns) c->pending_pj[die[i]] += retention_quantum_pj(c);   /* with the bins on it is booked where it is served */
            claimed[i] = 1;
            ++claims;
        }
        if (c->ret && !op) c->ret->disturb[retention_block_of(c, off)] += (uint32_t)np;
        s_ns[i] = s; cbs[i] = cb; eng[i] = e;
        if (op) { a_ns[i] = acc[i].issue_ns + xfer; post[i] = 0; }       /* program: data moves in first */
        else    { a_ns[i] = acc[i].issue_ns;        post[i] = xfer; }    /* read: data moves out after  */
        cnt[qu + 1]++;
    }

    /* per-queue lists in index order, then each sorted by (issue, index) */
    for (uint32_t r = 0; r < c->n_queues; ++r) cnt[r + 1] += cnt[r];
    {
        uint64_t *fill = (uint64_t *)malloc((size_t)c->n_queues * sizeof(uint64_t));
        if (!fill) { rc = HBFO_E_NOMEM; goto done; }
        memcpy(fill, cnt, (size_t)c->n_queues * sizeof(uint64_t));
        for (uint64_t i = 0; i < n; ++i) {
            if (st[i] != HBFO_ST_READY) continue;
            qent_t *e = &ent[fill[queue[i]]++];
            e->issue_ns = acc[i].issue_ns; e->idx = (uint32_t)i;
        }
        free(fill);
    }
    for (uint32_t r = 0; r < c->n_queues; ++r)
        qsort(ent + cnt[r], (size_t)(cnt[r + 1] - cnt[r]), sizeof(qent_t), cmp_qent);

    /* serve each queue, one access at a time */
    hbfo_die_stats_t *ds = (hbfo_die_stats_t *)calloc(c->n_dies, sizeof(hbfo_die_stats_t));
    if (!ds) { rc = HBFO_E_NOMEM; goto done; }
    for (uint64_t i = 0; i < n; ++i)
        if (st[i] == HBFO_ST_NATIVE) { completion_ns[i] = acc[i].issue_ns; stall_ns[i] = 0; }
    for (uint32_t r = 0; r < c->n_queues; ++r) {
        int64_t B = c->busy_until[r];
        for (uint64_t k = cnt[r]; k < cnt[r + 1]; ++k) {
            uint32_t i = ent[k].idx;
            int64_t start = a_ns[i] > B ? a_ns[i] : B;
            B = start + s_ns[i];
            int64_t done_ns = B + post[i];
            completion_ns[i] = done_ns;
            stall_ns[i] = done_ns - acc[i].issue_ns;
            hbfo_die_stats_t *d = &ds[die[i]];
            d->busy_ns += s_ns[i]; d->energy_pj += eng[i];
            if (c->bin_ns && claimed[i]) {                    /* the refresh quantum first, then the access's own service */
                const int64_t qns = retention_quantum_ns(c, q);
                ledger_event(c, die[i], start, qns, retention_quantum_pj(c));
                ledger_event(c, die[i], start + qns, s_ns[i] - qns, eng[i]);
            } else if (c->bin_ns) ledger_event(c, die[i], start, s_ns[i], eng[i]);
            if (acc[i].flags & 1u) { d->bytes_prog += cbs[i]; d->n_prog += 1; }
            else                   { d->bytes_read += cbs[i]; d->n_read += 1; }
            res.modeled_ns += stall_ns[i]; res.service_ns += s_ns[i];
            if (done_ns > res.max_completion_ns) res.max_completion_ns = done_ns;
            c->order[k] = i;
        }
        c->busy_until[r] = B;
    }
    c->order_count = n_ready;
    if (c->bus_busy) {
        /* second stage: per channel, the reads in the order the array finished them */
        bent_t *be = (bent_t *)malloc((n_ready ? n_ready : 1) * sizeof(bent_t));
        if (!be) { free(ds); rc = HBFO_E_NOMEM; goto done; }
        res.modeled_ns = 0; res.max_completion_ns = 0;
        for (uint32_t ch = 0; ch < c->cfg.channels; ++ch) {
            uint64_t m = 0;
            for (uint64_t i = 0; i < n; ++i)
                if (st[i] == HBFO_ST_READY && !(acc[i].flags & 1u) && die[i] / c->cfg.dies == ch) {
                    be[m].done_ns = completion_ns[i] - post[i]; be[m].idx = (uint32_t)i; ++m;
                }
            qsort(be, (size_t)m, sizeof(bent_t), cmp_bent);
            int64_t B = c->bus_busy[ch];
            for (uint64_t k = 0; k < m; ++k) {
                const uint32_t i = be[k].idx;
                int64_t start = be[k].done_ns > B ? be[k].done_ns : B;
                B = start + post[i];
                completion_ns[i] = B;
                stall_ns[i] = B - acc[i].issue_ns;
            }
            c->bus_busy[ch] = B;
        }
        free(be);
        for (uint64_t i = 0; i < n; ++i) {
            if (st[i] != HBFO_ST_READY) continue;
            res.modeled_ns += stall_ns[i];
            if (completion_ns[i] > res.max_completion_ns) res.max_completion_ns = completion_ns[i];
        }
    }
    if (!c->bin_ns) for (uint32_t d = 0; d < c->n_dies; ++d) c->pending_pj[d] += ds[d].energy_pj;
    if (die_stats) memcpy(die_stats, ds, c->n_dies * sizeof(hbfo_die_stats_t));
    free(ds);
    res.code = HBFO_OK; res.n_native = n_native; res.n_modeled = n_ready;
    c->last = res;
    if (c->ret) { c->ret->claimed += claims; retention_commit(c->ret); }

done:
    free(st); free(rg); free(queue); free(die); free(a_ns); free(s_ns); free(post); free(cbs); free(eng);
    free(cnt); free(ent); free(claimed);
    return rc;
}

/* ---- submit, page-granular (an extension the paper only implies: its back end is a flash simulator that
 * works in pages, Section "Design"; what follows is this build's definition) ---------------------------------
 * A modeled access is cut at page boundaries of the media into parts; part k covers the bytes of the access
 * that fall into its k-th page.  Every part is a request of its own: the batch of parts, listed in (access
 * index, part index) order, is served exactly as hbfo_submit_batch serves a batch of accesses.  So a part is
 * decoded by its own first byte (consecutive pages follow the stripe interleave onto other channels, dies and
 * planes), charged one page of array time and the transfer of its own bytes (whole granules), and queued on its
 * own queue in the order (issue time, access index, part index); and whatever else is switched on sees parts
 * too: a part's array interval is an event of the energy ledger on the part's die, a read part's transfer
 * queues on the bus of the part's channel in (array-done time, position in the list of parts) order, the parts
 * claim outstanding refresh quanta in list order, one each, and a read part disturbs the block of its own
 * page.  The access completes when its last part does.  Per-die statistics count parts (page operations); the
 * batch summary counts accesses.  An access that is not modeled is one part. */
int hbfo_submit_batch_paged(hbfo_ctx *c, const hbfo_access_t *acc, uint64_t n, int64_t *completion_ns,
                            int64_t *stall_ns, uint8_t *status, hbfo_die_stats_t *die_stats) {
    if (!c || (n && (!acc || !completion_ns || !stall_ns)) || n > 0xffffffffull) return HBFO_E_INVAL;
    hbfo_batch_result_t res; memset(&res, 0, sizeof(res));
    res.mode = c->mode; res.q_ppm = c->q_ppm;
    if (c->mode == HBFO_MODE_SHUTDOWN) { res.code = HBFO_E_LINK_SHUTDOWN; c->last = res; return res.code; }
    if (c->mode == HBFO_MODE_SEVERE)   { res.code = HBFO_E_THROTTLED;     c->last = res; return res.code; }
    c->order_count = 0;

    /* the accesses' own status; a fault refuses the batch before anything is split */
    uint8_t *st = (uint8_t *)malloc(n ? n : 1);
    int32_t *rg = (int32_t *)malloc((n ? n : 1) * sizeof(int32_t));
    if (!st || !rg) { free(st); free(rg); return HBFO_E_NOMEM; }
    uint64_t n_fault = 0, n_native = 0, n_ready = 0, n_parts = 0;
    const uint64_t pg = c->cfg.page_bytes;
    for (uint64_t i = 0; i < n; ++i) {
        st[i] = (uint8_t)hbfo_classify(c, &acc[i], &rg[i]);
        if (st[i] == HBFO_ST_NATIVE) { ++n_native; ++n_parts; }
        else if (st[i] == HBFO_ST_READY) {
            const range_t *r = &c->ranges[rg[i]];
            uint64_t off = r->media_offset + (acc[i].addr - r->base);
            n_parts += (off % pg + acc[i].bytes + pg - 1) / pg;
            ++n_ready;
        } else ++n_fault;
    }
    if (status) memcpy(status, st, n);
    if (n_fault) {
        if (die_stats) memset(die_stats, 0, c->n_dies * sizeof(hbfo_die_stats_t));
        memset(completion_ns, 0, n * sizeof(int64_t)); memset(stall_ns, 0, n * sizeof(int64_t));
        res.code = HBFO_E_ACCESS_FAULT; res.n_fault = n_fault; res.n_native = n_native;
        c->last = res; free(st); free(rg);
        return res.code;
    }
    if (n_parts > 0xffffffffull) { free(st); free(rg); return HBFO_E_INVAL; }

    /* the list of parts: records of their own, in (access, part) order */
    const uint64_t m = n_parts ? n_parts : 1;
    hbfo_access_t *part = (hbfo_access_t *)malloc(m * sizeof(hbfo_access_t));
    uint64_t *first = (uint64_t *)malloc((n + 1) * sizeof(uint64_t));   /* parts of access i: first[i] .. first[i + 1] - 1 */
    int64_t *pc = (int64_t *)malloc(m * sizeof(int64_t)), *ps = (int64_t *)malloc(m * sizeof(int64_t));
    int rc = HBFO_OK;
    if (!part || !first || !pc || !ps) { rc = HBFO_E_NOMEM; goto done; }
    uint64_t slot = 0;
    for (uint64_t i = 0; i < n; ++i) {
        first[i] = slot;
        if (st[i] != HBFO_ST_READY) { part[slot++] = acc[i]; continue; }
        const range_t *r = &c->ranges[rg[i]];
        const uint64_t off = r->media_offset + (acc[i].addr - r->base), end = off + acc[i].bytes;
        for (uint64_t lo = off; lo < end; ) {
            uint64_t hi = (lo / pg + 1) * pg;                 /* next page boundary */
            if (hi > end) hi = end;
            part[slot] = acc[i];
            part[slot].addr = acc[i].addr + (lo - off);
            part[slot].bytes = (uint32_t)(hi - lo);
            ++slot;
            lo = hi;
        }
    }
    first[n] = slot;

    rc = hbfo_submit_batch(c, part, n_parts, pc, ps, NULL, die_stats);
    c->order_count = 0;                                       /* the served order of parts is not reported */
    if (rc != HBFO_OK) {                                      /* refused as a whole, nothing changed */
        memset(completion_ns, 0, n * sizeof(int64_t)); memset(stall_ns, 0, n * sizeof(int64_t));
        goto done;
    }
    /* join: an access ends with the last of its parts */
    res = c->last;
    res.n_native = n_native; res.n_modeled = n_ready; res.modeled_ns = 0;
    for (uint64_t i = 0; i < n; ++i) {
        if (st[i] != HBFO_ST_READY) { completion_ns[i] = acc[i].issue_ns; stall_ns[i] = 0; continue; }
        int64_t last = pc[first[i]];
        for (uint64_t k = first[i] + 1; k < first[i + 1]; ++k) if (pc[k] > last) last = pc[k];
        completion_ns[i] = last;
        stall_ns[i] = last - acc[i].issue_ns;
        res.modeled_ns += stall_ns[i];
    }
    c->last = res;

done:
    free(st); free(rg); free(part); free(first); free(pc); free(ps);
    return rc;
}

int hbfo_last_result(hbfo_ctx *c, hbfo_batch_result_t *out) {
    if (!c || !out) return HBFO_E_INVAL;
    *out = c->last;
    return c->last.code;
}

int hbfo_last_order(hbfo_ctx *c, uint32_t *order, uint64_t cap, uint64_t *count) {
    if (!c || !count) return HBFO_E_INVAL;
    *count = c->order_count;
    if (order) {
        if (cap < c->order_count) return HBFO_E_INVAL;
        memcpy(order, c->order, c->order_count * sizeof(uint32_t));
    }
    return HBFO_OK;
}

int hbfo_get_busy_until(hbfo_ctx *c, int64_t *out, uint64_t cap) {
    if (!c || !out || cap < c->n_queues) return HBFO_E_INVAL;
    memcpy(out, c->busy_until, c->n_queues * sizeof(int64_t));
    return HBFO_OK;
}
int hbfo_get_pending_energy(hbfo_ctx *c, int64_t *out, uint64_t cap) {
    if (!c || !out || cap < c->n_dies) return HBFO_E_INVAL;
    memcpy(out, c->pending_pj, c->n_dies * sizeof(int64_t));
    return HBFO_OK;
}
int hbfo_get_temps(hbfo_ctx *c, double *out, uint64_t cap) {
    if (!c || !c->thermal || !out || cap < c->n_cells) return HBFO_E_INVAL;
    memcpy(out, c->T, c->n_cells * sizeof(double));
    return HBFO_OK;
}
int hbfo_set_temps(hbfo_ctx *c, const double *in, uint64_t count) {
    if (!c || !c->thermal || !in || count != c->n_cells) return HBFO_E_INVAL;
    memcpy(c->T, in, c->n_cells * sizeof(double));
    return HBFO_OK;
}

/* ---- thermal step (Design D3, Eq. 1) ------------------------------------------------------- */

int64_t hbfo_quantise_mk(double t_c) { return (int64_t)floor(t_c * 1000.0 + 0.5); }   /* round half up */

int32_t hbfo_next_mode(hbfo_ctx *c, int32_t mode, int64_t t) {
    const int64_t rtt = hbfo_quantise_mk((double)c->cfg.rtt_c), ltt = hbfo_quantise_mk((double)c->cfg.ltt_c);
    const int64_t stt = hbfo_quantise_mk((double)c->cfg.stt_c), shut = hbfo_quantise_mk((double)c->cfg.shutdown_c);
    if (mode == HBFO_MODE_SHUTDOWN) return HBFO_MODE_SHUTDOWN;            /* absorbing */
    if (t >= shut) return HBFO_MODE_SHUTDOWN;
    switch (mode) {
    case HBFO_MODE_NORMAL:
        if (t >= stt) return HBFO_MODE_SEVERE;
        if (t >= ltt) return HBFO_MODE_LIGHT;
        return HBFO_MODE_NORMAL;
    case HBFO_MODE_LIGHT:
        if (t >= stt) return HBFO_MODE_SEVERE;
        if (t <= rtt) return HBFO_MODE_NORMAL;
        return HBFO_MODE_LIGHT;
    case HBFO_MODE_SEVERE:
        if (t <= rtt) return HBFO_MODE_NORMAL;
        if (t <= ltt) return HBFO_MODE_LIGHT;
        return HBFO_MODE_SEVERE;
    default: return mode;
    }
}

int hbfo_thermal_step(hbfo_ctx *c, int64_t dt_ns, const float *ext_power_w, uint32_t n_ext,
                      double *temps_out, double hot_c_out[3]) {
    if (!c || !c->thermal || dt_ns <= 0) return HBFO_E_INVAL;
    if (n_ext != 0 && (n_ext != c->cfg.n_regions || !ext_power_w)) return HBFO_E_INVAL;
    const uint32_t H = c->cfg.grid_h, W = c->cfg.grid_w, NR = c->cfg.n_regions;
    const double dt_s = (double)dt_ns * 1e-9;
    const double dt_sub = dt_s / (double)c->cfg.n_sub;
    if (dt_sub > c->euler_limit_s) return HBFO_E_INVAL;                    /* explicit step would be unstable */
    const double amb = (double)c->cfg.ambient_c;

    if (c->bin_ns) {                                          /* the step is the bin the thermal clock stands in */
        if (dt_ns != c->bin_ns) return HBFO_E_INVAL;
        int64_t *row = c->ledger + (size_t)(c->cur_bin % c->n_bins) * c->n_dies;
        for (uint32_t d = 0; d < c->n_dies; ++d) { c->pending_pj[d] += row[d]; row[d] = 0; }
        c->cur_bin += 1;
    }
    /* power map: energy of the window / window length + idle + external, spread over the region */
    double *Pr = (double *)calloc(NR, sizeof(double));
    if (!Pr) return HBFO_E_NOMEM;
    for (uint32_t d = 0; d < c->n_dies; ++d)
        Pr[c->die_region[d]] += ((double)c->pending_pj[d] * 1e-12) / dt_s;
    for (uint32_t g = 0; g < NR; ++g) {
        Pr[g] += c->region_idle_w[g];
        if (n_ext) Pr[g] += (double)ext_power_w[g];
    }
    for (size_t i = 0; i < c->n_cells; ++i) {
        int32_t g = c->cell_region[i];
        c->P[i] = g >= 0 ? Pr[g] / c->region_cells[g] : 0.0;
    }
    free(Pr);
    memset(c->pending_pj, 0, c->n_dies * sizeof(int64_t));

    /* explicit Euler, every cell from the previous substep's field */
    for (uint32_t k = 0; k < c->cfg.n_sub; ++k) {
        for (uint32_t y = 0; y < H; ++y) for (uint32_t x = 0; x < W; ++x) {
            size_t i = (size_t)y * W + x;
            double Ti = c->T[i], flow = 0.0;
            if (x + 1 < W) flow += c->Gx[i]     * (Ti - c->T[i + 1]);
            if (x > 0)     flow += c->Gx[i - 1] * (Ti - c->T[i - 1]);
            if (y + 1 < H) flow += c->Gy[i]     * (Ti - c->T[i + W]);
            if (y > 0)     flow += c->Gy[i - W] * (Ti - c->T[i - W]);
            c->Tn[i] = Ti + dt_sub / c->C[i] * (c->P[i] - flow - c->Gs[i] * (Ti - amb));
        }
        double *t = c->T; c->T = c->Tn; c->Tn = t;
    }

    /* hotspots per medium; the HBF one drives the controller */
    double hot[3] = { -INFINITY, -INFINITY, -INFINITY };
    for (size_t i = 0; i < c->n_cells; ++i) {
        int32_t g = c->cell_region[i];
        if (g < 0) continue;
        int32_t k = c->region_kind[g];
        int slot = k == HBFO_KIND_HBF ? 0 : k == HBFO_KIND_HBM ? 1 : k == HBFO_KIND_GPU ? 2 : -1;
        if (slot >= 0 && c->T[i] > hot[slot]) hot[slot] = c->T[i];
    }
    for (int k = 0; k < 3; ++k) if (hot[k] == -INFINITY) hot[k] = amb;
    c->mode = hbfo_next_mode(c, c->mode, hbfo_quantise_mk(hot[0]));
    if (c->mode == HBFO_MODE_NORMAL) c->q_ppm = 1000000;
    else if (c->mode == HBFO_MODE_LIGHT) c->q_ppm = c->cfg.q_light_ppm;
    if (temps_out) memcpy(temps_out, c->T, c->n_cells * sizeof(double));
    if (hot_c_out) { hot_c_out[0] = hot[0]; hot_c_out[1] = hot[1]; hot_c_out[2] = hot[2]; }
    return HBFO_OK;
}

/* ---- reduced-order thermal model (Eq. 2): x' = A x + B p + b,  T = C x + D p + d, with x the state BEFORE
 * the update.  Plain loops in double; matrices row-major. */
struct hbfo_rom {
    uint32_t n, m, o;
    double *A, *B, *b, *C, *D, *d, *x, *xn;
};

static double *dup_f64(const double *src, size_t n) {
    double *p = (double *)malloc((n ? n : 1) * sizeof(double));
    if (p && src) memcpy(p, src, n * sizeof(double));
    else if (p) memset(p, 0, (n ? n : 1) * sizeof(double));
    return p;
}

int hbfo_rom_destroy(hbfo_rom *r) {
    if (!r) return HBFO_E_INVAL;
    free(r->A); free(r->B); free(r->b); free(r->C); free(r->D); free(r->d); free(r->x); free(r->xn); free(r);
    return HBFO_OK;
}

int hbfo_rom_create(uint32_t n_states, uint32_t n_inputs, uint32_t n_outputs, const double *A, const double *B,
                    const double *b, const double *C, const double *D, const double *d, hbfo_rom **out) {
    if (!out || !n_states || !n_inputs || !n_outputs || !A || !B || !C) return HBFO_E_INVAL;
    hbfo_rom *r = (hbfo_rom *)calloc(1, sizeof(hbfo_rom));
    if (!r) return HBFO_E_NOMEM;
    r->n = n_states; r->m = n_inputs; r->o = n_outputs;
    r->A = dup_f64(A, (size_t)n_states * n_states); r->B = dup_f64(B, (size_t)n_states * n_inputs);
    r->b = dup_f64(b, n_states); r->C = dup_f64(C, (size_t)n_outputs * n_states);
    r->D = dup_f64(D, (size_t)n_outputs * n_inputs); r->d = dup_f64(d, n_outputs);
    r->x = dup_f64(NULL, n_states); r->xn = dup_f64(NULL, n_states);
    if (!r->A || !r->B || !r->b || !r->C || !r->D || !r->d || !r->x || !r->xn) { hbfo_rom_destroy(r); return HBFO_E_NOMEM; }
    *out = r;
    return HBFO_OK;
}

int hbfo_rom_reset(hbfo_rom *r) { if (!r) return HBFO_E_INVAL; memset(r->x, 0, r->n * sizeof(double)); return HBFO_OK; }

/* n_steps steps: power [n_steps][n_inputs] in, temps_out [n_steps][n_outputs] out */
int hbfo_rom_step(hbfo_rom *r, const double *power, uint32_t n_steps, double *temps_out) {
    if (!r || !power || !temps_out) return HBFO_E_INVAL;
    for (uint32_t k = 0; k < n_steps; ++k) {
        const double *p = power + (size_t)k * r->m;
        double *T = temps_out + (size_t)k * r->o;
        for (uint32_t i = 0; i < r->o; ++i) {
            double acc = r->d[i];
            for (uint32_t j = 0; j < r->n; ++j) acc += r->C[(size_t)i * r->n + j] * r->x[j];
            for (uint32_t j = 0; j < r->m; ++j) acc += r->D[(size_t)i * r->m + j] * p[j];
            T[i] = acc;
        }
        for (uint32_t i = 0; i < r->n; ++i) {
            double acc = r->b[i];
            for (uint32_t j = 0; j < r->n; ++j) acc += r->A[(size_t)i * r->n + j] * r->x[j];
            for (uint32_t j = 0; j < r->m; ++j) acc += r->B[(size_t)i * r->m + j] * p[j];
            r->xn[i] = acc;
        }
        double *t = r->x; r->x = r->xn; r->xn = t;
    }
    return HBFO_OK;
}

int hbfo_rom_get_state(hbfo_rom *r, double *out, uint64_t cap) {
    if (!r || !out || cap < r->n) return HBFO_E_INVAL;
    memcpy(out, r->x, r->n * sizeof(double));
    return HBFO_OK;
}

/* ---- thermal step on the reduced-order model (the paper's run-time configuration: the service simulation runs on
 * the fitted model, Section "Evaluation", not on the full operator).  Same power vector as hbfo_thermal_step
 * (window energy / dt + idle + external, one entry per region), one step of the model, then the controller on the
 * hottest output of each medium (output_kind[i] = HBFO_KIND_* of output i).  The grid field is not advanced. */
int hbfo_thermal_step_rom(hbfo_ctx *c, hbfo_rom *r, const int32_t *output_kind, int64_t dt_ns, const float *ext_power_w,
                          uint32_t n_ext, double hot_c_out[3]) {
    if (!c || !c->thermal || !r || !output_kind || dt_ns <= 0 || r->m != c->cfg.n_regions) return HBFO_E_INVAL;
    if (n_ext != 0 && (n_ext != c->cfg.n_regions || !ext_power_w)) return HBFO_E_INVAL;
    const uint32_t NR = c->cfg.n_regions;
    const double dt_s = (double)dt_ns * 1e-9;
    if (c->bin_ns) {
        if (dt_ns != c->bin_ns) return HBFO_E_INVAL;
        int64_t *row = c->ledger + (size_t)(c->cur_bin % c->n_bins) * c->n_dies;
        for (uint32_t d = 0; d < c->n_dies; ++d) { c->pending_pj[d] += row[d]; row[d] = 0; }
        c->cur_bin += 1;
    }
    double *Pr = (double *)calloc(NR, sizeof(double)), *T = (double *)calloc(r->o, sizeof(double));
    if (!Pr || !T) { free(Pr); free(T); return HBFO_E_NOMEM; }
    for (uint32_t d = 0; d < c->n_dies; ++d)
        Pr[c->die_region[d]] += ((double)c->pending_pj[d] * 1e-12) / dt_s;
    for (uint32_t g = 0; g < NR; ++g) {
        Pr[g] += c->region_idle_w[g];
        if (n_ext) Pr[g] += (double)ext_power_w[g];
    }
    memset(c->pending_pj, 0, c->n_dies * sizeof(int64_t));
    int rc = hbfo_rom_step(r, Pr, 1, T);
    if (rc == HBFO_OK) {
        double hot[3] = {-1e300, -1e300, -1e300};
        for (uint32_t i = 0; i < r->o; ++i) {
            int slot = output_kind[i] == HBFO_KIND_HBF ? 0 : output_kind[i] == HBFO_KIND_HBM ? 1 : output_kind[i] == HBFO_KIND_GPU ? 2 : -1;
            if (slot >= 0 && T[i] > hot[slot]) hot[slot] = T[i];
        }
        for (int k = 0; k < 3; ++k) if (hot[k] == -1e300) hot[k] = (double)c->cfg.ambient_c;
        c->mode = hbfo_next_mode(c, c->mode, hbfo_quantise_mk(hot[0]));
        if (c->mode == HBFO_MODE_NORMAL) c->q_ppm = 1000000;
        else if (c->mode == HBFO_MODE_LIGHT) c->q_ppm = c->cfg.q_light_ppm;
        if (hot_c_out) { hot_c_out[0] = hot[0]; hot_c_out[1] = hot[1]; hot_c_out[2] = hot[2]; }
    }
    free(Pr); free(T);
    return rc;
}
