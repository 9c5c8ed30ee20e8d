// Host shell of libhbf.so: argument validation, context and range bookkeeping, launches.
// No step of the service model runs here; the host only checks arguments and enqueues kernels.
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "hbf_dev.cuh"

using namespace hbf;

namespace {

struct HostRange { uint64_t base, length, media_offset; uint32_t perms, kind, stream_tag, id; };

struct StateHeader {            // hbf_get_state / hbf_set_state blob header
    uint32_t magic, version, n_queues, n_dies, n_cells; int32_t mode; int64_t q_ppm; int32_t poisoned, cur;
    // version 2: what else the context has switched on, each with the sizes that fix its section's length
    uint32_t flags, n_channels;          // kStateBus | kStateBins | kStateRetention
    int64_t bin_ns, cur_bin; uint32_t n_bins, pad;
    uint64_t ret_blocks, ret_plan_cap;
};
constexpr uint32_t kStateBus = 1u, kStateBins = 2u, kStateRetention = 4u;
constexpr uint32_t kStateMagic = 0x48424631u;   // "HBF1"

}  // namespace

struct hbf_rom;
struct hbf_ctx {
    hbf_config_t cfg{};
    cudaStream_t stream = nullptr;
    int device = 0, sm_count = 148;
    ModelParams mp{};
    std::vector<HostRange> ranges;
    uint32_t next_range_id = 0;
    int32_t path = HBF_PATH_AUTO;
    bool terminal = false;           // a shutdown result has been observed
    // device state
    RangeSnap *d_ranges = nullptr; ModelParams *d_mp = nullptr; DevState *d_state = nullptr;
    BatchCtrl *d_ctrl = nullptr; hbf_batch_result_t *d_result = nullptr;
    int64_t *d_busy = nullptr, *d_busy_stage = nullptr, *d_pending = nullptr; hbf_die_stats_t *d_stats_stage = nullptr;
    hbf_batch_result_t *h_result = nullptr;      // pinned
    TileBalanceHost bal;                         // tile sizes of the in-order path from the times earlier batches left
    // thermal steps on a reduced-order model instead of the grid (off while rom == nullptr)
    hbf_rom *rom = nullptr; int64_t rom_dt_ns = 0; int32_t *d_rom_kind = nullptr; double *d_rom_p = nullptr, *d_rom_T = nullptr;
    // channel bus as a second queued stage (off while d_bus_busy == nullptr)
    int64_t *d_bus_busy = nullptr; BatchCtrl *d_bus_ctrl = nullptr;
    // time-bin energy ledger (off while bin_ns == 0)
    int64_t bin_ns = 0, cur_bin = 0; uint32_t n_bins = 0; unsigned long long *d_ledger = nullptr;
    // retention, refresh and wear (off while ret_on == false)
    bool ret_on = false; RetDev ret{}; hbf_retention_config_t ret_cfg{};
    float *h_hot = nullptr;                      // pinned [3]
    float *h_ext = nullptr;                      // pinned [n_regions]
    std::vector<float> last_ext;                 // the external powers the device holds (empty: none sent yet)
    bool submitted = false;
    uint32_t spin_limit = kSpinLimit, test_stage = 0, test_tile = 0;   // bounded device-side waits (test support: hbf_debug_wait_test)
    bool profiling = false; cudaEvent_t ev[kProfEvents] = {}; cudaEvent_t ev_th[2] = {}; bool ev_made = false;
    bool prof_submit = false, prof_thermal = false, prof_inorder = false, inorder_ok = false;
    // thermal
    bool thermal = false; ThermalDev td{}; int cur = 0; double euler_limit_s = 0.0; bool thermal_generic = false;
    std::vector<void *> owned;
    // host-buffer pipeline of hbf_submit_host (allocated at its first use, sized for the largest chunk seen)
    struct HostPipe {
        uint64_t chunk = 0; size_t ws_bytes = 0;
        hbf_access_t *acc[2] = {}; int64_t *comp[2] = {}, *stall[2] = {}; hbf_die_stats_t *stats = nullptr, *total = nullptr; void *ws = nullptr;
        hbf_batch_result_t *d_sum = nullptr, *h_sum = nullptr;          // the chunks' summaries added up: device, and pinned
        cudaStream_t s_in = nullptr, s_out = nullptr;
        cudaEvent_t arrived[2] = {}, served[2] = {}, read[2] = {}, start = nullptr;
        bool made = false;
    } pipe;
};

#define CK(expr) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) return HBF_E_CUDA; } while (0)

static Div64 make_div64_host(uint64_t d) {       // same construction as the device helper
    Div64 r; r.magic = 0; r.shift = 0; r.pow2 = 0;
    if ((d & (d - 1)) == 0) { r.pow2 = 1; while ((1ull << r.shift) < d) ++r.shift; return r; }
    uint32_t l = 0; while (l < 64 && (1ull << l) < d) ++l;
    r.magic = (uint64_t)(((unsigned __int128)1 << (63 + l)) / d) + 1ull; r.shift = l - 1;
    return r;
}

// the context's device state, kernels' attributes and stream belong to the device it was created on
static bool on_own_device(const hbf_ctx *c) { int d = -1; return cudaGetDevice(&d) == cudaSuccess && d == c->device; }

static bool is_pow2(uint64_t v) { return v && !(v & (v - 1)); }
static uint32_t log2u(uint64_t v) { uint32_t s = 0; while ((1ull << s) < v) ++s; return s; }

template <typename T>
static int dev_copy(hbf_ctx *c, T **dst, const void *src, size_t count) {
    void *p = nullptr;
    if (cudaMalloc(&p, std::max<size_t>(count, 1) * sizeof(T)) != cudaSuccess) return HBF_E_NOMEM;
    c->owned.push_back(p);
    if (src) { if (cudaMemcpy(p, src, count * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) return HBF_E_CUDA; }
    else if (cudaMemset(p, 0, std::max<size_t>(count, 1) * sizeof(T)) != cudaSuccess) return HBF_E_CUDA;
    *dst = static_cast<T *>(p);
    return HBF_OK;
}

static int publish_ranges(hbf_ctx *c) {
    RangeSnap snap; memset(&snap, 0, sizeof(snap));
    std::vector<HostRange> sorted = c->ranges;
    std::sort(sorted.begin(), sorted.end(), [](const HostRange &a, const HostRange &b) { return a.base < b.base; });
    snap.count = (uint32_t)sorted.size();
    for (size_t i = 0; i < sorted.size(); ++i) {
        snap.base[i] = sorted[i].base; snap.length[i] = sorted[i].length;
        snap.media_offset[i] = sorted[i].media_offset; snap.perms[i] = sorted[i].perms;
    }
    // ordered after every batch already enqueued, before every later one
    CK(cudaMemcpyAsync(c->d_ranges, &snap, sizeof(snap), cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

// ---- retention, refresh and wear (Design D4) ----------------------------------------------------------------
static int retention_clear(hbf_ctx *c) {
    const RetDev &r = c->ret;
    CK(cudaMemsetAsync(r.damage, 0, r.n_blocks * 8, c->stream));
    CK(cudaMemsetAsync(r.disturb, 0, r.n_blocks * 4, c->stream));
    CK(cudaMemsetAsync(r.pec, 0, r.n_blocks * 4, c->stream));
    CK(cudaMemsetAsync(r.epoch_of, 0, r.n_blocks * 4, c->stream));
    CK(cudaMemsetAsync(r.worn, 0, r.n_blocks, c->stream));
    CK(cudaMemsetAsync(r.die_claims, 0, (size_t)c->mp.n_dies * 4, c->stream));
    CK(cudaMemsetAsync(r.st, 0, sizeof(RetState), c->stream));
    return HBF_OK;
}

extern "C" {

// ---- reduced-order thermal model (Eq. 2) ----------------------------------------------------------------------
struct hbf_rom {
    uint32_t n = 0, m = 0, o = 0;
    cudaStream_t stream = nullptr;
    double *d_all = nullptr;             // A, B, b, C, D, d, x in one allocation
    double *A = nullptr, *B = nullptr, *b = nullptr, *C = nullptr, *D = nullptr, *d = nullptr, *x = nullptr;
};

int hbf_rom_create(uint32_t n_states, uint32_t n_inputs, uint32_t n_outputs, const double *A, const double *B, const double *b,
                   const double *C, const double *D, const double *d, void *cuda_stream, hbf_rom **out) {
    if (!out || !n_states || !n_inputs || !n_outputs || !A || !B || !C) return HBF_E_INVAL;
    if ((size_t)(2 * n_states + n_inputs) * sizeof(double) > 40u * 1024u) return HBF_E_INVAL;   // the step keeps x, x' and p in shared memory
    const size_t n = n_states, m = n_inputs, o = n_outputs;
    const size_t total = n * n + n * m + n + o * n + o * m + o + n;
    std::vector<double> h(total, 0.0);
    double *p = h.data();
    auto put = [&](const double *src, size_t cnt) { if (src) memcpy(p, src, cnt * sizeof(double)); double *at = p; p += cnt; return at - h.data(); };
    const size_t oA = put(A, n * n), oB = put(B, n * m), ob = put(b, n), oC = put(C, o * n), oD = put(D, o * m), od = put(d, o), ox = put(nullptr, n);
    hbf_rom *r = new (std::nothrow) hbf_rom();
    if (!r) return HBF_E_NOMEM;
    r->n = n_states; r->m = n_inputs; r->o = n_outputs; r->stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMalloc(&r->d_all, total * sizeof(double)) != cudaSuccess) { delete r; return HBF_E_NOMEM; }
    if (cudaMemcpyAsync(r->d_all, h.data(), total * sizeof(double), cudaMemcpyHostToDevice, r->stream) != cudaSuccess ||
        cudaStreamSynchronize(r->stream) != cudaSuccess) { cudaFree(r->d_all); delete r; return HBF_E_CUDA; }
    r->A = r->d_all + oA; r->B = r->d_all + oB; r->b = r->d_all + ob; r->C = r->d_all + oC; r->D = r->d_all + oD; r->d = r->d_all + od;
    r->x = r->d_all + ox;
    *out = r;
    return HBF_OK;
}

int hbf_rom_destroy(hbf_rom *r) {
    if (!r) return HBF_E_INVAL;
    cudaStreamSynchronize(r->stream);
    cudaFree(r->d_all);
    delete r;
    return HBF_OK;
}

int hbf_rom_reset(hbf_rom *r) {
    if (!r) return HBF_E_INVAL;
    CK(cudaMemsetAsync(r->x, 0, r->n * sizeof(double), r->stream));
    return HBF_OK;
}

int hbf_rom_step(hbf_rom *r, const double *d_power, uint32_t n_steps, double *d_temps_out) {
    if (!r || !d_power || !d_temps_out) return HBF_E_INVAL;
    if (n_steps == 0) return HBF_OK;
    CK(launch_rom_steps(r->n, r->m, r->o, r->A, r->B, r->b, r->C, r->D, r->d, r->x, d_power, n_steps, d_temps_out, r->stream));
    return HBF_OK;
}

int hbf_rom_get_state(hbf_rom *r, double *host_out, uint64_t cap) {
    if (!r || !host_out || cap < r->n) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, r->x, r->n * sizeof(double), cudaMemcpyDeviceToHost, r->stream));
    CK(cudaStreamSynchronize(r->stream));
    return HBF_OK;
}

uint32_t hbf_rom_outputs(const hbf_rom *r) { return r ? r->o : 0u; }

int hbf_attach_rom(hbf_ctx *c, hbf_rom *r, const int32_t *output_kind, int64_t dt_ns) {
    if (!c || !c->thermal) return HBF_E_INVAL;
    CK(cudaStreamSynchronize(c->stream));
    if (!r) { c->rom = nullptr; return HBF_OK; }               // back to the grid
    if (!output_kind || dt_ns <= 0 || r->m != c->td.n_regions || r->stream != c->stream) return HBF_E_INVAL;
    if (c->d_rom_kind) { cudaFree(c->d_rom_kind); c->d_rom_kind = nullptr; }
    if (c->d_rom_p) { cudaFree(c->d_rom_p); c->d_rom_p = nullptr; }
    if (cudaMalloc(&c->d_rom_kind, r->o * sizeof(int32_t)) != cudaSuccess) return HBF_E_NOMEM;
    if (cudaMalloc(&c->d_rom_p, ((size_t)r->m + r->o) * sizeof(double)) != cudaSuccess) return HBF_E_NOMEM;
    c->d_rom_T = c->d_rom_p + r->m;
    CK(cudaMemcpyAsync(c->d_rom_kind, output_kind, r->o * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    c->rom = r; c->rom_dt_ns = dt_ns;
    return HBF_OK;
}

int hbf_get_rom_temps(hbf_ctx *c, double *host_out, uint64_t cap) {
    if (!c || !c->rom || !host_out || cap < c->rom->o) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, c->d_rom_T, c->rom->o * sizeof(double), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

const char *hbf_strerror(int code) {
    switch (code) {
    case HBF_OK: return "ok";
    case HBF_E_INVAL: return "invalid argument";
    case HBF_E_RANGE_OVERLAP: return "range overlaps a registered range";
    case HBF_E_RANGE_FULL: return "range table full";
    case HBF_E_CAPACITY: return "range exceeds media capacity";
    case HBF_E_WORKSPACE: return "workspace too small or misaligned";
    case HBF_E_CUDA: return "CUDA runtime error";
    case HBF_E_ACCESS_FAULT: return "batch refused: fail-closed access";
    case HBF_E_THROTTLED: return "throttled: new reservations withheld";
    case HBF_E_LINK_SHUTDOWN: return "link shutdown";
    case HBF_E_TIMEOUT: return "bounded device wait expired";
    case HBF_E_NOMEM: return "out of memory";
    default: return "unknown";
    }
}

int hbf_destroy(hbf_ctx *c) {
    if (!c) return HBF_E_INVAL;
    cudaStreamSynchronize(c->stream);
    for (void *p : c->owned) cudaFree(p);
    if (c->ev_made) { for (auto &e : c->ev) cudaEventDestroy(e); for (auto &e : c->ev_th) cudaEventDestroy(e); }
    if (c->h_result) cudaFreeHost(c->h_result);
    if (c->bal.pinned) cudaFreeHost(c->bal.pinned);
    if (c->d_ledger) cudaFree(c->d_ledger);
    if (c->d_bus_busy) cudaFree(c->d_bus_busy);
    if (c->d_bus_ctrl) cudaFree(c->d_bus_ctrl);
    if (c->d_rom_kind) cudaFree(c->d_rom_kind);
    if (c->d_rom_p) cudaFree(c->d_rom_p);
    if (c->h_hot) cudaFreeHost(c->h_hot);
    if (c->h_ext) cudaFreeHost(c->h_ext);
    if (c->pipe.made) {
        hbf_ctx::HostPipe &p = c->pipe;
        cudaStreamSynchronize(p.s_in); cudaStreamSynchronize(p.s_out);
        for (int k = 0; k < 2; ++k) { cudaFree(p.acc[k]); cudaFree(p.comp[k]); cudaFree(p.stall[k]); cudaEventDestroy(p.arrived[k]); cudaEventDestroy(p.served[k]); cudaEventDestroy(p.read[k]); }
        cudaFree(p.stats); cudaFree(p.total); cudaFree(p.ws); cudaEventDestroy(p.start);
        if (p.h_sum) cudaFreeHost(p.h_sum);
        cudaFree(p.d_sum);
        cudaStreamDestroy(p.s_in); cudaStreamDestroy(p.s_out);
    }
    delete c;
    return HBF_OK;
}

int hbf_create(const hbf_config_t *cfg, void *cuda_stream, hbf_ctx **out) {
    if (!cfg || !out) return HBF_E_INVAL;
    if (!cfg->channels || !cfg->dies || !cfg->planes) return HBF_E_INVAL;
    if (!is_pow2(cfg->page_bytes) || !is_pow2(cfg->stripe_bytes) || cfg->stripe_bytes < cfg->page_bytes) return HBF_E_INVAL;
    if (!is_pow2(cfg->read_granule) || !is_pow2(cfg->prog_granule) || cfg->queue_level > 1) return HBF_E_INVAL;
    if (cfg->t_read_ns <= 0 || cfg->t_prog_ns <= 0 || !cfg->chan_bytes_per_us) return HBF_E_INVAL;
    if (cfg->e_cmd_read_pj < 0 || cfg->e_byte_read_pj < 0 || cfg->e_cmd_prog_pj < 0 || cfg->e_byte_prog_pj < 0) return HBF_E_INVAL;
    if (cfg->q_light_ppm < 1 || cfg->q_light_ppm > 1000000) return HBF_E_INVAL;
    const uint64_t nd = (uint64_t)cfg->channels * cfg->dies;
    const uint64_t nq = cfg->queue_level == 0 ? nd * cfg->planes : nd;
    if (nq > 65536 || nd > 65536) return HBF_E_INVAL;

    hbf_ctx *c = new (std::nothrow) hbf_ctx();
    if (!c) return HBF_E_NOMEM;
    c->cfg = *cfg; c->stream = static_cast<cudaStream_t>(cuda_stream);
    int rc = HBF_OK;
    auto fail = [&](int code) { hbf_destroy(c); return code; };
    if (cudaGetDevice(&c->device) != cudaSuccess) return fail(HBF_E_CUDA);
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) return fail(HBF_E_CUDA);
    c->sm_count = prop.multiProcessorCount;

    ModelParams &mp = c->mp;
    mp.channels = cfg->channels; mp.dies = cfg->dies; mp.planes = cfg->planes;
    mp.n_queues = (uint32_t)nq; mp.n_dies = (uint32_t)nd;
    mp.page_shift = log2u(cfg->page_bytes); mp.stripe_shift = log2u(cfg->stripe_bytes);
    mp.pages_per_stripe_shift = mp.stripe_shift - mp.page_shift;
    mp.queue_level = cfg->queue_level;
    mp.pow2_geom = is_pow2(cfg->channels) && is_pow2(cfg->dies) && is_pow2(cfg->planes);
    mp.ch_shift = log2u(cfg->channels); mp.die_shift = log2u(cfg->dies); mp.plane_shift = log2u(cfg->planes);
    mp.read_gran_shift = log2u(cfg->read_granule); mp.prog_gran_shift = log2u(cfg->prog_granule);
    mp.t_read_ns = cfg->t_read_ns; mp.t_prog_ns = cfg->t_prog_ns; mp.chan_bytes_per_us = cfg->chan_bytes_per_us;
    mp.e_cmd_read_pj = cfg->e_cmd_read_pj; mp.e_byte_read_pj = cfg->e_byte_read_pj;
    mp.e_cmd_prog_pj = cfg->e_cmd_prog_pj; mp.e_byte_prog_pj = cfg->e_byte_prog_pj;

    mp.div_chan = make_div64_host(cfg->chan_bytes_per_us);
    {   // the in-order path packs the transfer time of an access into 31 bits and keeps per-queue state in shared memory
        const unsigned __int128 worst = ((unsigned __int128)0xffffffffull + std::max(cfg->read_granule, cfg->prog_granule)) * 1000u;
        c->inorder_ok = nq <= kInMaxQueues && worst / cfg->chan_bytes_per_us < ((unsigned __int128)1 << 31) &&
                        inorder_serve_smem((uint32_t)nd) + 8u * 1024u <= 227u * 1024u;
    }
    {   // transfer times of the small charged sizes, looked up instead of divided (every charged size is a multiple of its granule)
        const uint32_t g = std::min(mp.read_gran_shift, mp.prog_gran_shift);
        std::vector<uint32_t> tab(1025);
        bool fits = true;
        for (uint32_t k = 0; k <= 1024; ++k) {
            const unsigned __int128 x = (((unsigned __int128)k << g) * 1000u + cfg->chan_bytes_per_us - 1) / cfg->chan_bytes_per_us;
            if (x >> 31) fits = false;
            tab[k] = (uint32_t)x;
        }
        mp.xfer_tab = nullptr; mp.xfer_tab_shift = g; mp.xfer_tab_max_cb = 0;
        if (fits && g < 21) {
            uint32_t *d = nullptr;
            if ((rc = dev_copy(c, &d, tab.data(), tab.size()))) return fail(rc);
            mp.xfer_tab = d; mp.xfer_tab_max_cb = 1024u << g;
        }
    }
    DevState st0; st0.mode = HBF_MODE_NORMAL; st0.poisoned = 0; st0.q_ppm = 1000000;
    st0.spin_limit = c->spin_limit; st0.test_stage = c->test_stage; st0.test_tile = c->test_tile; st0.pad = 0;
    if ((rc = dev_copy(c, &c->d_ranges, nullptr, 1))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_mp, &mp, 1))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_state, &st0, 1))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_ctrl, nullptr, 1))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_result, nullptr, 1))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_busy, nullptr, nq))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_busy_stage, nullptr, nq))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_pending, nullptr, nd))) return fail(rc);
    if ((rc = dev_copy(c, &c->d_stats_stage, nullptr, nd))) return fail(rc);
    if (cudaMallocHost(&c->h_result, sizeof(hbf_batch_result_t)) != cudaSuccess) return fail(HBF_E_NOMEM);
    memset(c->h_result, 0, sizeof(hbf_batch_result_t));
    if (cudaMallocHost(&c->h_hot, 3 * sizeof(float)) != cudaSuccess) return fail(HBF_E_NOMEM);
    if ((rc = dev_copy(c, &c->bal.dev, nullptr, 1))) return fail(rc);
    if (cudaMallocHost(&c->bal.pinned, sizeof(TileBalance)) != cudaSuccess) return fail(HBF_E_NOMEM);
    memset(c->bal.pinned, 0, sizeof(TileBalance));

    c->thermal = cfg->cell_C != nullptr;
    if (c->thermal) {
        if (!cfg->grid_h || !cfg->grid_w || !cfg->n_sub || !cfg->n_regions || !cfg->cell_Gx || !cfg->cell_Gy ||
            !cfg->cell_Gsink || !cfg->cell_region || !cfg->die_region || !cfg->region_kind || !cfg->region_idle_w)
            return fail(HBF_E_INVAL);
        if (!(cfg->rtt_c < cfg->ltt_c && cfg->ltt_c < cfg->stt_c && cfg->stt_c < cfg->shutdown_c)) return fail(HBF_E_INVAL);
        const uint32_t H = cfg->grid_h, W = cfg->grid_w, NR = cfg->n_regions;
        const size_t nc = (size_t)H * W;
        if (nc > (1u << 30)) return fail(HBF_E_INVAL);
        std::vector<float> inv_cells(NR, 0.0f); std::vector<double> cells(NR, 0.0);
        double lim = INFINITY;
        for (uint32_t y = 0; y < H; ++y) for (uint32_t x = 0; x < W; ++x) {
            const size_t i = (size_t)y * W + x;
            if (!(cfg->cell_C[i] > 0.0f) || cfg->cell_Gx[i] < 0.0f || cfg->cell_Gy[i] < 0.0f || cfg->cell_Gsink[i] < 0.0f) return fail(HBF_E_INVAL);
            const int32_t g = cfg->cell_region[i];
            if (g >= (int32_t)NR) return fail(HBF_E_INVAL);
            if (g >= 0) cells[g] += 1.0;
            double gs = cfg->cell_Gsink[i];
            if (x + 1 < W) gs += cfg->cell_Gx[i];
            if (x > 0) gs += cfg->cell_Gx[i - 1];
            if (y + 1 < H) gs += cfg->cell_Gy[i];
            if (y > 0) gs += cfg->cell_Gy[i - W];
            if (gs > 0.0) lim = std::min(lim, (double)cfg->cell_C[i] / gs);
        }
        c->euler_limit_s = lim;
        std::vector<int32_t> ptr(NR + 1, 0), list(nd);
        for (uint64_t d = 0; d < nd; ++d) {
            const int32_t g = cfg->die_region[d];
            if (g < 0 || g >= (int32_t)NR || cells[g] == 0.0) return fail(HBF_E_INVAL);
            ptr[g + 1]++;
        }
        for (uint32_t g = 0; g < NR; ++g) { ptr[g + 1] += ptr[g]; inv_cells[g] = cells[g] > 0.0 ? (float)(1.0 / cells[g]) : 0.0f; }
        { std::vector<int32_t> fill(ptr.begin(), ptr.end() - 1);
          for (uint64_t d = 0; d < nd; ++d) list[fill[cfg->die_region[d]]++] = (int32_t)d; }
        ThermalDev &t = c->td;
        t.H = H; t.W = W; t.n_regions = NR; t.n_dies = (uint32_t)nd; t.n_sub = cfg->n_sub; t.ambient_c = cfg->ambient_c;
        auto mk = [](float v) { return (int64_t)std::floor((double)v * 1000.0 + 0.5); };
        t.rtt_mk = mk(cfg->rtt_c); t.ltt_mk = mk(cfg->ltt_c); t.stt_mk = mk(cfg->stt_c); t.shut_mk = mk(cfg->shutdown_c);
        t.q_light_ppm = cfg->q_light_ppm;
        float *p;
        int32_t *q;
        double *dp;
        if ((rc = dev_copy(c, &p, cfg->cell_C, nc))) return fail(rc); t.C = p;
        if ((rc = dev_copy(c, &p, cfg->cell_Gx, nc))) return fail(rc); t.Gx = p;
        if ((rc = dev_copy(c, &p, cfg->cell_Gy, nc))) return fail(rc); t.Gy = p;
        if ((rc = dev_copy(c, &p, cfg->cell_Gsink, nc))) return fail(rc); t.Gs = p;
        if ((rc = dev_copy(c, &q, cfg->cell_region, nc))) return fail(rc); t.cell_region = q;
        if ((rc = dev_copy(c, &q, cfg->die_region, nd))) return fail(rc); t.die_region = q;
        if ((rc = dev_copy(c, &q, cfg->region_kind, NR))) return fail(rc); t.region_kind = q;
        if ((rc = dev_copy(c, &p, cfg->region_idle_w, NR))) return fail(rc); t.region_idle_w = p;
        if ((rc = dev_copy(c, &p, inv_cells.data(), NR))) return fail(rc); t.region_inv_cells = p;
        if ((rc = dev_copy(c, &q, ptr.data(), NR + 1))) return fail(rc); t.region_die_ptr = q;
        if ((rc = dev_copy(c, &q, list.data(), nd))) return fail(rc); t.region_die_list = q;
        if ((rc = dev_copy(c, &t.theta[0], nullptr, nc))) return fail(rc);
        if ((rc = dev_copy(c, &t.theta[1], nullptr, nc))) return fail(rc);
        if ((rc = dev_copy(c, &t.comp, nullptr, nc))) return fail(rc);
        if ((rc = dev_copy(c, &t.P, nullptr, nc))) return fail(rc);
        if ((rc = dev_copy(c, &dp, nullptr, NR))) return fail(rc); t.region_power = dp;
        if ((rc = dev_copy(c, &t.ext_power, nullptr, NR))) return fail(rc);
        if ((rc = dev_copy(c, &t.hot, nullptr, 3))) return fail(rc);
        if (cudaMallocHost(&c->h_ext, NR * sizeof(float)) != cudaSuccess) return fail(HBF_E_NOMEM);
        // the descriptor keeps no pointer into the caller's arrays
        c->cfg.cell_C = c->cfg.cell_Gx = c->cfg.cell_Gy = c->cfg.cell_Gsink = c->cfg.region_idle_w = nullptr;
        c->cfg.cell_region = c->cfg.die_region = c->cfg.region_kind = nullptr;
    }
    if (cudaDeviceSynchronize() != cudaSuccess) return fail(HBF_E_CUDA);
    *out = c;
    return HBF_OK;
}

int hbf_register_range(hbf_ctx *c, uint64_t base, uint64_t length, uint32_t perms, uint32_t kind,
                       uint32_t stream_tag, uint64_t media_offset, uint32_t *out_id) {
    if (!c || length == 0 || (perms & ~3u) || perms == 0 || kind > 1) return HBF_E_INVAL;
    if (base + length < base || media_offset + length < media_offset) return HBF_E_INVAL;
    if (c->cfg.capacity_bytes && media_offset + length > c->cfg.capacity_bytes) return HBF_E_CAPACITY;
    if (c->ranges.size() >= HBF_MAX_RANGES) return HBF_E_RANGE_FULL;
    for (const HostRange &r : c->ranges)
        if (base < r.base + r.length && r.base < base + length) return HBF_E_RANGE_OVERLAP;
    HostRange r{base, length, media_offset, perms, kind, stream_tag, c->next_range_id++};
    c->ranges.push_back(r);
    if (out_id) *out_id = r.id;
    return publish_ranges(c);
}

int hbf_clear_ranges(hbf_ctx *c) {
    if (!c) return HBF_E_INVAL;
    c->ranges.clear();
    return publish_ranges(c);
}

size_t hbf_workspace_bytes(const hbf_ctx *c, uint64_t n) {
    if (!c) return 0;
    return workspace_layout(n, c->mp.n_queues, nullptr, nullptr, c->d_bus_busy ? 1 : 0);
}

int hbf_set_thermal_path(hbf_ctx *c, int32_t generic_only) {
    if (!c) return HBF_E_INVAL;
    c->thermal_generic = generic_only != 0;
    return HBF_OK;
}

int hbf_set_path(hbf_ctx *c, int32_t path) {
    if (!c || path < 0 || path > 3) return HBF_E_INVAL;
    c->path = path;
    return HBF_OK;
}

int hbf_get_tile_times(hbf_ctx *c, uint32_t *records_out, uint32_t *ns_out, uint32_t cap, uint32_t *count) {
    if (!c || !count) return HBF_E_INVAL;
    CK(cudaStreamSynchronize(c->stream));
    const TileBalance &r = *c->bal.pinned;
    uint32_t n = 0;
    while (n < kInBalMax && r.claim[n] != 0u && r.claim[n] == r.claim[0]) ++n;
    *count = n;
    if (records_out && ns_out) {
        if (cap < n) return HBF_E_INVAL;
        for (uint32_t t = 0; t < n; ++t) { records_out[t] = r.len[t]; ns_out[t] = r.ns[t]; }
    }
    return HBF_OK;
}

int hbf_set_tile_balance(hbf_ctx *c, int32_t on) {
    if (!c) return HBF_E_INVAL;
    c->bal.on = on != 0;
    if (c->bal.pinned) memset(c->bal.pinned, 0, sizeof(TileBalance));      // (measurements start over)
    c->bal.depth = 0; c->bal.depth_seen = 0;
    return HBF_OK;
}

int hbf_set_head_entries(hbf_ctx *c, uint32_t entries) {
    if (!c || entries > 6u) return HBF_E_INVAL;
    c->bal.depth_fixed = entries;
    return HBF_OK;
}

// Everything a batch of records goes through once its arguments are in place: the claim window (retention), the submit
// path, the energy ledger, read disturb / commits, the channel-bus stage.  Shared by hbf_submit_batch (the caller's
// accesses) and hbf_submit_batch_paged (the list of parts).
static int serve_records(hbf_ctx *c, SubmitArgs &a) {
    a.ranges = c->d_ranges; a.mp_dev = c->d_mp; a.mp = c->mp; a.state = c->d_state; a.ctrl = c->d_ctrl; a.result = c->d_result;
    a.busy = c->d_busy; a.busy_stage = c->d_busy_stage; a.pending = c->d_pending; a.stats_stage = c->d_stats_stage;
    a.path = c->path; a.sm_count = c->sm_count; a.inorder_ok = c->inorder_ok ? 1 : 0;
    if (c->ranges.size() == 1) {
        const HostRange &r = c->ranges[0];
        a.fast.base = r.base; a.fast.length = r.length; a.fast.media_offset = r.media_offset; a.fast.perms = r.perms; a.fast.on = 1u;
    }
    a.binned = c->bin_ns != 0; a.bus_on = c->d_bus_busy ? 1 : 0;
    a.bal = &c->bal;
    if (c->ret_on) {                                         // how far the outstanding refresh quanta reach into this batch
        CK(launch_ret_window(a.acc, a.n, c->d_ranges, c->ret, c->sm_count, c->stream));
        a.claim_limit = &c->ret.st->claim_limit; a.die_claims = c->ret.die_claims; a.ret = &c->ret;
    }
    CK(launch_submit(a, c->stream));
    if (a.binned) {
        const int64_t page = (int64_t)1 << c->mp.page_shift;
        const int64_t quantum_pj = c->mp.e_cmd_read_pj + c->mp.e_byte_read_pj * page + c->mp.e_cmd_prog_pj + c->mp.e_byte_prog_pj * page;
        CK(launch_energy_bins(a.acc, a.n, a.completion, c->d_ranges, c->d_mp, c->d_ctrl, c->d_result, c->d_ledger, c->bin_ns,
                              c->n_bins, c->cur_bin, c->sm_count, a.claim_limit, quantum_pj, c->stream));
    }
    if (c->ret_on)                                           // read disturb, commits, the claimed energy (after the ledger: it needs the claim limit)
        CK(launch_ret_close(a.acc, a.n, c->d_ranges, c->d_mp, c->mp, c->d_result, c->d_pending, a.binned, c->ret, c->sm_count, c->stream));
    if (c->d_bus_busy)                                       // after the ledger: its events are the array intervals
        CK(launch_bus_stage(a, c->d_bus_ctrl, c->d_bus_busy, c->stream));
    return HBF_OK;
}

int hbf_submit_batch(hbf_ctx *c, const hbf_access_t *d_acc, uint64_t n, int64_t *d_completion_ns,
                     int64_t *d_stall_ns, uint8_t *d_status, hbf_die_stats_t *d_die_stats,
                     void *d_workspace, size_t workspace_bytes) {
    if (!c || !on_own_device(c)) return HBF_E_INVAL;
    if (c->terminal) return HBF_E_LINK_SHUTDOWN;
    if (n > HBF_MAX_BATCH) return HBF_E_INVAL;
    if (n && (!d_acc || !d_completion_ns || !d_stall_ns)) return HBF_E_INVAL;
    if ((reinterpret_cast<uintptr_t>(d_acc) & 7u) || (reinterpret_cast<uintptr_t>(d_completion_ns) & 7u) ||
        (reinterpret_cast<uintptr_t>(d_stall_ns) & 7u) || (reinterpret_cast<uintptr_t>(d_die_stats) & 7u)) return HBF_E_INVAL;
    SubmitArgs a{};
    const size_t need = workspace_layout(n, c->mp.n_queues, &a.ws, d_workspace, c->d_bus_busy ? 1 : 0);
    if (!d_workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return HBF_E_WORKSPACE;
    a.acc = d_acc; a.n = n; a.completion = d_completion_ns; a.stall = d_stall_ns; a.status = d_status; a.die_stats = d_die_stats;
    c->prof_inorder = c->profiling && n > 0 && c->inorder_ok && (c->path == HBF_PATH_AUTO || c->path == HBF_PATH_INORDER);
    a.ev = c->profiling ? c->ev : nullptr;
    c->prof_submit = c->profiling;
    const int rc = serve_records(c, a);
    if (rc != HBF_OK) return rc;
    c->submitted = true;
    return HBF_OK;
}

// Host-buffer submit: the batch is cut into chunks; the copy-in of chunk k+1, the service of chunk k (hbf_submit_batch)
// and the read-back of chunk k-1 run on three streams, so the link moves both ways while the kernels run.
static int host_pipe_prepare(hbf_ctx *c, uint64_t chunk) {
    hbf_ctx::HostPipe &p = c->pipe;
    if (!p.made) {
        CK(cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking));
        CK(cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking));
        for (int k = 0; k < 2; ++k) {
            CK(cudaEventCreateWithFlags(&p.arrived[k], cudaEventDisableTiming));
            CK(cudaEventCreateWithFlags(&p.served[k], cudaEventDisableTiming));
            CK(cudaEventCreateWithFlags(&p.read[k], cudaEventDisableTiming));
        }
        CK(cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming));
        if (cudaMalloc(&p.stats, (size_t)c->mp.n_dies * sizeof(hbf_die_stats_t)) != cudaSuccess) return HBF_E_NOMEM;
        if (cudaMalloc(&p.total, (size_t)c->mp.n_dies * sizeof(hbf_die_stats_t)) != cudaSuccess) return HBF_E_NOMEM;
        if (cudaMalloc(&p.d_sum, sizeof(hbf_batch_result_t)) != cudaSuccess) return HBF_E_NOMEM;
        if (cudaMallocHost(&p.h_sum, sizeof(hbf_batch_result_t)) != cudaSuccess) return HBF_E_NOMEM;
        p.made = true;
    }
    const size_t ws_need = hbf_workspace_bytes(c, chunk);
    if (chunk > p.chunk || ws_need > p.ws_bytes) {
        CK(cudaStreamSynchronize(c->stream)); CK(cudaStreamSynchronize(p.s_in)); CK(cudaStreamSynchronize(p.s_out));
        for (int k = 0; k < 2; ++k) {
            cudaFree(p.acc[k]); cudaFree(p.comp[k]); cudaFree(p.stall[k]); p.acc[k] = nullptr; p.comp[k] = p.stall[k] = nullptr;
            if (cudaMalloc(&p.acc[k], chunk * sizeof(hbf_access_t)) != cudaSuccess || cudaMalloc(&p.comp[k], chunk * 8) != cudaSuccess ||
                cudaMalloc(&p.stall[k], chunk * 8) != cudaSuccess) { p.chunk = 0; return HBF_E_NOMEM; }
        }
        cudaFree(p.ws); p.ws = nullptr;
        if (cudaMalloc(&p.ws, ws_need) != cudaSuccess) { p.chunk = 0; p.ws_bytes = 0; return HBF_E_NOMEM; }
        p.chunk = chunk; p.ws_bytes = ws_need;
    }
    return HBF_OK;
}

int hbf_submit_host(hbf_ctx *c, const hbf_access_t *h_acc, uint64_t n, int64_t *h_completion_ns, int64_t *h_stall_ns,
                    hbf_die_stats_t *h_die_stats, uint64_t chunk, hbf_batch_result_t *summary_out) {
    if (!c || !on_own_device(c)) return HBF_E_INVAL;
    if (c->terminal) return HBF_E_LINK_SHUTDOWN;
    if (n && (!h_acc || !h_completion_ns || !h_stall_ns)) return HBF_E_INVAL;
    if (chunk == 0) chunk = 4000000;
    chunk = std::min<uint64_t>(std::min<uint64_t>(chunk, HBF_MAX_BATCH), std::max<uint64_t>(n, 1));
    int rc = host_pipe_prepare(c, chunk);
    if (rc != HBF_OK) return rc;
    hbf_ctx::HostPipe &p = c->pipe;
    cudaStream_t main = c->stream;
    CK(cudaEventRecord(p.start, main));                      // the side streams begin behind what the context has enqueued so far
    CK(cudaStreamWaitEvent(p.s_in, p.start, 0)); CK(cudaStreamWaitEvent(p.s_out, p.start, 0));
    CK(cudaMemsetAsync(p.total, 0, (size_t)c->mp.n_dies * sizeof(hbf_die_stats_t), main));
    bool served[2] = {false, false}, read[2] = {false, false};
    size_t k = 0;
    for (uint64_t lo = 0; lo < n; lo += chunk, ++k) {
        const uint64_t m = std::min<uint64_t>(chunk, n - lo);
        const int s = (int)(k & 1);
        if (served[s]) CK(cudaStreamWaitEvent(p.s_in, p.served[s], 0));   // the slot's records have been read by the chunk before last
        CK(cudaMemcpyAsync(p.acc[s], h_acc + lo, m * sizeof(hbf_access_t), cudaMemcpyHostToDevice, p.s_in));
        CK(cudaEventRecord(p.arrived[s], p.s_in));
        CK(cudaStreamWaitEvent(main, p.arrived[s], 0));
        if (read[s]) CK(cudaStreamWaitEvent(main, p.read[s], 0));         // the slot's results have left
        rc = hbf_submit_batch(c, p.acc[s], m, p.comp[s], p.stall[s], nullptr, p.stats, p.ws, p.ws_bytes);
        if (rc != HBF_OK) break;
        CK(launch_add_stats(p.total, p.stats, c->mp.n_dies, main));       // (a refused chunk leaves zeros)
        CK(launch_add_result(p.d_sum, c->d_result, k == 0 ? 1 : 0, main));
        CK(cudaEventRecord(p.served[s], main)); served[s] = true;
        CK(cudaStreamWaitEvent(p.s_out, p.served[s], 0));
        CK(cudaMemcpyAsync(h_completion_ns + lo, p.comp[s], m * 8, cudaMemcpyDeviceToHost, p.s_out));
        CK(cudaMemcpyAsync(h_stall_ns + lo, p.stall[s], m * 8, cudaMemcpyDeviceToHost, p.s_out));
        CK(cudaEventRecord(p.read[s], p.s_out)); read[s] = true;
    }
    for (int s = 0; s < 2; ++s) if (read[s]) CK(cudaStreamWaitEvent(main, p.read[s], 0));
    if (rc != HBF_OK) { cudaStreamSynchronize(main); return rc; }
    if (k) CK(cudaMemcpyAsync(p.h_sum, p.d_sum, sizeof(hbf_batch_result_t), cudaMemcpyDeviceToHost, main));
    if (h_die_stats) CK(cudaMemcpyAsync(h_die_stats, p.total, (size_t)c->mp.n_dies * sizeof(hbf_die_stats_t), cudaMemcpyDeviceToHost, main));
    CK(cudaStreamSynchronize(main));                         // results, totals and the chunks' summaries are on the host
    hbf_batch_result_t sum; memset(&sum, 0, sizeof(sum));
    if (k) sum = *p.h_sum;
    if (sum.code == HBF_E_LINK_SHUTDOWN) c->terminal = true;
    if (summary_out) *summary_out = sum;
    return sum.code;
}

size_t hbf_workspace_bytes_paged(const hbf_ctx *c, uint64_t n, uint64_t parts_capacity) {
    if (!c) return 0;
    return paged_layout(n, std::max<uint64_t>(parts_capacity, n), c->mp.n_queues, nullptr, nullptr, c->d_bus_busy ? 1 : 0);
}

int hbf_submit_batch_paged(hbf_ctx *c, const hbf_access_t *d_acc, uint64_t n, uint64_t parts_capacity,
                           int64_t *d_completion_ns, int64_t *d_stall_ns, uint8_t *d_status, hbf_die_stats_t *d_die_stats,
                           void *d_workspace, size_t workspace_bytes) {
    if (!c) return HBF_E_INVAL;
    if (n == 0)                                             // nothing to split: the ordinary path reports the empty batch
        return hbf_submit_batch(c, d_acc, 0, d_completion_ns, d_stall_ns, d_status, d_die_stats, d_workspace, workspace_bytes);
    if (!on_own_device(c)) return HBF_E_INVAL;
    if (c->terminal) return HBF_E_LINK_SHUTDOWN;
    if (n > HBF_MAX_BATCH) return HBF_E_INVAL;
    if (!d_acc || !d_completion_ns || !d_stall_ns) return HBF_E_INVAL;
    if ((reinterpret_cast<uintptr_t>(d_acc) & 7u) || (reinterpret_cast<uintptr_t>(d_completion_ns) & 7u) ||
        (reinterpret_cast<uintptr_t>(d_stall_ns) & 7u) || (reinterpret_cast<uintptr_t>(d_die_stats) & 7u)) return HBF_E_INVAL;
    const uint64_t capacity = std::min<uint64_t>(std::max<uint64_t>(parts_capacity, n), HBF_MAX_BATCH);
    PagedWorkspace pw{};
    const int with_bus = c->d_bus_busy ? 1 : 0;
    const size_t need = paged_layout(n, capacity, c->mp.n_queues, &pw, d_workspace, with_bus);
    if (!d_workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(d_workspace) & 255u)) return HBF_E_WORKSPACE;
    // how many parts: the one point where the host waits for the device inside a submit
    CK(launch_paged_count(d_acc, n, c->d_ranges, c->d_mp, pw, c->stream));
    unsigned long long *h_total = reinterpret_cast<unsigned long long *>(c->h_result);     // pinned, free between calls
    CK(cudaMemcpyAsync(h_total, pw.total, sizeof(unsigned long long), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    const uint64_t total = *h_total;
    if (total > capacity) return HBF_E_WORKSPACE;            // nothing has changed: the caller may come back with more room
    FastRange fast{};
    if (c->ranges.size() == 1) {
        const HostRange &r = c->ranges[0];
        fast.base = r.base; fast.length = r.length; fast.media_offset = r.media_offset; fast.perms = r.perms; fast.on = 1u;
    }
    CK(launch_paged_expand(d_acc, n, c->d_ranges, c->d_mp, fast, c->mp.page_shift, capacity, pw, c->sm_count, c->stream));
    // the list of parts is a batch of records like any other: the ledger, the bus stage and retention, when on, see parts
    SubmitArgs a{};
    workspace_layout(total, c->mp.n_queues, &a.ws, pw.inner, with_bus);
    a.acc = pw.parts; a.n = total; a.completion = pw.part_completion; a.stall = pw.part_stall; a.status = pw.part_status;
    a.die_stats = d_die_stats;
    c->prof_inorder = false; c->prof_submit = false;
    a.ev = nullptr;
    const int rc = serve_records(c, a);
    if (rc != HBF_OK) return rc;
    CK(launch_paged_join(d_acc, n, pw, c->d_result, d_completion_ns, d_stall_ns, d_status, c->sm_count, c->stream));
    c->submitted = true;
    return HBF_OK;
}

int hbf_enable_channel_bus(hbf_ctx *c) {
    if (!c) return HBF_E_INVAL;
    if (c->d_bus_busy) return HBF_OK;
    CK(cudaStreamSynchronize(c->stream));
    int64_t *b = nullptr; BatchCtrl *bc = nullptr;
    if (cudaMalloc(&b, (size_t)c->mp.channels * 8) != cudaSuccess) return HBF_E_NOMEM;
    if (cudaMalloc(&bc, sizeof(BatchCtrl)) != cudaSuccess) { cudaFree(b); return HBF_E_NOMEM; }
    c->d_bus_busy = b; c->d_bus_ctrl = bc;
    CK(cudaMemsetAsync(b, 0, (size_t)c->mp.channels * 8, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_bus_busy_until(hbf_ctx *c, int64_t *host_out, uint64_t cap) {
    if (!c || !c->d_bus_busy || !host_out || cap < c->mp.channels) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, c->d_bus_busy, (size_t)c->mp.channels * 8, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_enable_retention(hbf_ctx *c, const hbf_retention_config_t *cfg) {
    if (!c || !cfg || c->ret_on) return HBF_E_INVAL;
    if (!cfg->pages_per_block || !cfg->blocks_per_plane || !cfg->blocks_per_zone ||
        cfg->blocks_per_plane % cfg->blocks_per_zone != 0 || !cfg->max_pec) return HBF_E_INVAL;
    if (!(cfg->l_ref_s > 0.0) || !(cfg->t_ref_c > -273.15) || !(cfg->ea_ev >= 0.0) || !(cfg->accel > 0.0) ||
        !(cfg->lead_threshold > 0.0)) return HBF_E_INVAL;
    const uint64_t nb = (uint64_t)c->mp.n_dies * c->mp.planes * cfg->blocks_per_plane;
    if (nb * cfg->pages_per_block > 0xffffffffull) return HBF_E_INVAL;      // a quantum id is 32 bits
    CK(cudaStreamSynchronize(c->stream));
    RetDev r{};
    r.ppb = cfg->pages_per_block; r.bpp = cfg->blocks_per_plane; r.bpz = cfg->blocks_per_zone; r.max_pec = cfg->max_pec;
    r.disturb_limit = cfg->disturb_limit; r.n_regions = c->thermal ? c->td.n_regions : 1u;
    r.div_ppb = make_div64_host(cfg->pages_per_block); r.div_bpp = make_div64_host(cfg->blocks_per_plane);
    {
        const uint64_t ppb = cfg->pages_per_block, bpp = cfg->blocks_per_plane;
        r.pow2 = ((ppb & (ppb - 1)) == 0 && (bpp & (bpp - 1)) == 0 && ppb * bpp < (1ull << 32) && c->mp.pow2_geom && c->mp.stripe_shift < 32) ? 1u : 0u;
        r.ppb_shift = 0;
        while ((1ull << r.ppb_shift) < ppb) ++r.ppb_shift;
    }
    r.accel = cfg->accel; r.lead = cfg->lead_threshold; r.l_ref_s = cfg->l_ref_s; r.t_ref_k = cfg->t_ref_c + 273.15;
    r.ea_over_kb = cfg->ea_ev / 8.617333262e-5;                             // Boltzmann constant in eV/K
    r.n_blocks = nb; r.plan_cap = nb * cfg->pages_per_block;
    int rc;
    if ((rc = dev_copy<double>(c, &r.damage, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.disturb, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.pec, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.epoch_of, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint8_t>(c, &r.worn, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<unsigned long long>(c, &r.last_pos, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.plan, nullptr, r.plan_cap)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.rank, nullptr, nb)) != HBF_OK) return rc;
    if ((rc = dev_copy<unsigned long long>(c, &r.die_len, nullptr, c->mp.n_dies)) != HBF_OK) return rc;
    if ((rc = dev_copy<unsigned long long>(c, &r.chan_len, nullptr, c->mp.channels)) != HBF_OK) return rc;
    r.chan_tab = nullptr;
    if (c->mp.channels <= kRetTabChannels) {
        const size_t C = c->mp.channels;
        if ((rc = dev_copy<uint32_t>(c, &r.chan_tab, nullptr, 2 * C + 1 + C * C)) != HBF_OK) return rc;
    }
    if ((rc = dev_copy<uint32_t>(c, &r.die_claims, nullptr, c->mp.n_dies)) != HBF_OK) return rc;
    if ((rc = dev_copy<uint32_t>(c, &r.tile_count, nullptr, (HBF_MAX_BATCH + 1023) / 1024 + 1)) != HBF_OK) return rc;
    if ((rc = dev_copy<double>(c, &r.rate, nullptr, r.n_regions)) != HBF_OK) return rc;
    if ((rc = dev_copy<double>(c, &r.region_temp, nullptr, r.n_regions)) != HBF_OK) return rc;
    if ((rc = dev_copy<int>(c, &r.region_max, nullptr, r.n_regions)) != HBF_OK) return rc;
    if ((rc = dev_copy<RetState>(c, &r.st, nullptr, 1)) != HBF_OK) return rc;
    c->ret = r; c->ret_cfg = *cfg; c->ret_on = true;
    return HBF_OK;
}

int hbf_retention_advance(hbf_ctx *c, int64_t dt_ns, const double *region_temp_c) {
    if (!c || !c->ret_on || dt_ns < 0) return HBF_E_INVAL;
    if (!region_temp_c && (!c->thermal || c->rom)) return HBF_E_INVAL;      // no field to read the temperatures from
    if (region_temp_c)                                                      // pageable source: staged before the call returns
        CK(cudaMemcpyAsync(c->ret.region_temp, region_temp_c, c->ret.n_regions * sizeof(double), cudaMemcpyHostToDevice, c->stream));
    CK(launch_ret_advance(c->ret, c->mp, c->thermal ? &c->td : nullptr, c->thermal ? c->td.theta[c->cur] : nullptr,
                          c->thermal ? c->td.die_region : nullptr, region_temp_c ? 1 : 0, dt_ns, c->sm_count, c->stream));
    return HBF_OK;
}

int hbf_retention_decay(hbf_ctx *c, int64_t idle_ns) {
    if (!c || !c->ret_on || idle_ns < 0) return HBF_E_INVAL;
    CK(launch_ret_decay(c->ret, c->mp, c->d_state, idle_ns, c->sm_count, c->stream));
    return HBF_OK;
}

int hbf_get_retention_blocks(hbf_ctx *c, double *damage, uint32_t *disturb, uint32_t *pec, uint32_t *epoch, uint64_t cap) {
    if (!c || !c->ret_on || cap < c->ret.n_blocks) return HBF_E_INVAL;
    const RetDev &r = c->ret;
    if (damage) CK(cudaMemcpyAsync(damage, r.damage, r.n_blocks * 8, cudaMemcpyDeviceToHost, c->stream));
    if (disturb) CK(cudaMemcpyAsync(disturb, r.disturb, r.n_blocks * 4, cudaMemcpyDeviceToHost, c->stream));
    if (pec) CK(cudaMemcpyAsync(pec, r.pec, r.n_blocks * 4, cudaMemcpyDeviceToHost, c->stream));
    if (epoch) CK(cudaMemcpyAsync(epoch, r.epoch_of, r.n_blocks * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

static int retention_state(hbf_ctx *c, RetState *out) {
    CK(cudaMemcpyAsync(out, c->ret.st, sizeof(RetState), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_retention_plan(hbf_ctx *c, uint32_t *quanta, uint64_t cap, uint64_t *count) {
    if (!c || !c->ret_on || !count) return HBF_E_INVAL;
    RetState s; int rc = retention_state(c, &s);
    if (rc != HBF_OK) return rc;
    const uint64_t mark = s.claimed + s.decayed, m = s.planned - mark;
    *count = m;
    if (!quanta) return HBF_OK;
    if (cap < m) return HBF_E_INVAL;
    const uint64_t first = mark % c->ret.plan_cap, head = std::min<uint64_t>(m, c->ret.plan_cap - first);   // the ring may wrap once
    if (head) CK(cudaMemcpyAsync(quanta, c->ret.plan + first, head * 4, cudaMemcpyDeviceToHost, c->stream));
    if (m > head) CK(cudaMemcpyAsync(quanta + head, c->ret.plan, (m - head) * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_retention_totals(hbf_ctx *c, hbf_retention_totals_t *out) {
    if (!c || !c->ret_on || !out) return HBF_E_INVAL;
    RetState s; int rc = retention_state(c, &s);
    if (rc != HBF_OK) return rc;
    std::vector<uint32_t> ep(c->ret.n_blocks);
    CK(cudaMemcpyAsync(ep.data(), c->ret.epoch_of, c->ret.n_blocks * 4, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    out->n_blocks = c->ret.n_blocks; out->planned = s.planned; out->claimed = s.claimed; out->decayed = s.decayed;
    out->commits = s.commits; out->worn_blocks = s.worn_blocks; out->epoch = s.epoch; out->pad = 0;
    out->waiting_blocks = 0;
    for (uint32_t e : ep) if (e) out->waiting_blocks += 1;
    return HBF_OK;
}

int hbf_enable_energy_bins(hbf_ctx *c, int64_t bin_ns, uint32_t n_bins) {
    if (!c || bin_ns <= 0 || n_bins == 0) return HBF_E_INVAL;
    CK(cudaStreamSynchronize(c->stream));
    unsigned long long *l = nullptr;
    if (cudaMalloc(&l, (size_t)n_bins * c->mp.n_dies * 8) != cudaSuccess) return HBF_E_NOMEM;
    if (c->d_ledger) cudaFree(c->d_ledger);
    c->d_ledger = l; c->bin_ns = bin_ns; c->n_bins = n_bins; c->cur_bin = 0;
    CK(cudaMemsetAsync(c->d_ledger, 0, (size_t)n_bins * c->mp.n_dies * 8, c->stream));
    CK(cudaMemsetAsync(c->d_pending, 0, c->mp.n_dies * sizeof(int64_t), c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_energy_bins(hbf_ctx *c, int64_t *host_out, uint64_t cap, int64_t *first_bin) {
    if (!c || !c->d_ledger || !host_out || cap < (uint64_t)c->n_bins * c->mp.n_dies) return HBF_E_INVAL;
    const size_t row = (size_t)c->mp.n_dies * 8;
    for (uint32_t k = 0; k < c->n_bins; ++k)                // row k of the output is bin cur_bin + k
        CK(cudaMemcpyAsync(host_out + (size_t)k * c->mp.n_dies, c->d_ledger + (size_t)((c->cur_bin + k) % c->n_bins) * c->mp.n_dies,
                           row, cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (first_bin) *first_bin = c->cur_bin;
    return HBF_OK;
}

int hbf_last_result(hbf_ctx *c, hbf_batch_result_t *host_out) {
    if (!c || !host_out) return HBF_E_INVAL;
    if (!c->submitted) { memset(host_out, 0, sizeof(*host_out)); return HBF_OK; }
    CK(cudaMemcpyAsync(c->h_result, c->d_result, sizeof(hbf_batch_result_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    *host_out = *c->h_result;
    if (host_out->code == HBF_E_LINK_SHUTDOWN) c->terminal = true;
    return host_out->code;
}

int hbf_queue_order(hbf_ctx *c, const void *d_workspace, uint64_t n, uint32_t *d_order, uint64_t *count) {
    if (!c || !d_workspace || !d_order || !count) return HBF_E_INVAL;
    Workspace ws;
    workspace_layout(n, c->mp.n_queues, &ws, const_cast<void *>(d_workspace));
    CK(launch_queue_order(c->d_ctrl, ws, d_order, n, c->stream));
    BatchCtrl hc;
    CK(cudaMemcpyAsync(&hc, c->d_ctrl, sizeof(hc), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (hc.code != HBF_OK || hc.inorder_used) return HBF_E_INVAL;
    *count = hc.n_ready;
    return HBF_OK;
}

int hbf_thermal_step(hbf_ctx *c, int64_t dt_ns, const float *ext_power_w, uint32_t n_ext, float *d_temps_out, float *hot_c_out) {
    if (!c || !c->thermal || dt_ns <= 0 || !on_own_device(c)) return HBF_E_INVAL;
    if (n_ext != 0 && (n_ext != c->td.n_regions || !ext_power_w)) return HBF_E_INVAL;
    const double dt_sub = (double)dt_ns * 1e-9 / (double)c->td.n_sub;
    // every refusal comes before the first enqueue: a refused call leaves the ledger, the clock and the stream as they were
    if (!c->rom && dt_sub > c->euler_limit_s) return HBF_E_INVAL;
    if (c->bin_ns && dt_ns != c->bin_ns) return HBF_E_INVAL;
    if (c->rom && (dt_ns != c->rom_dt_ns || d_temps_out)) return HBF_E_INVAL;
    // pageable source: the runtime stages the bytes before returning, so the caller's array is free at once.  A loop that
    // steps with the same powers every time (the usual case) sends them once.
    if (n_ext && (c->last_ext.size() != n_ext || memcmp(c->last_ext.data(), ext_power_w, n_ext * sizeof(float)) != 0)) {
        CK(cudaMemcpyAsync(c->td.ext_power, ext_power_w, n_ext * sizeof(float), cudaMemcpyHostToDevice, c->stream));
        c->last_ext.assign(ext_power_w, ext_power_w + n_ext);
    }
    if (c->bin_ns) {                                         // the step is the bin the thermal clock stands in
        CK(launch_take_bin(c->d_ledger + (size_t)(c->cur_bin % c->n_bins) * c->mp.n_dies, c->d_pending, c->mp.n_dies, c->stream));
        c->cur_bin += 1;
    }
    if (c->profiling) CK(cudaEventRecord(c->ev_th[0], c->stream));
    if (c->rom) {                                            // the attached model stands in for the grid
        CK(launch_rom_power(c->td, c->d_pending, dt_ns, n_ext != 0, c->d_rom_p, c->stream));
        { const int rc_ = hbf_rom_step(c->rom, c->d_rom_p, 1, c->d_rom_T); if (rc_ != HBF_OK) return rc_; }
        CK(launch_rom_controller(c->td, c->d_rom_T, c->d_rom_kind, hbf_rom_outputs(c->rom), c->d_state, c->stream));
    } else {
        CK(launch_thermal_step(c->td, c->d_state, c->d_pending, dt_ns, n_ext != 0, d_temps_out, &c->cur, c->thermal_generic ? 1 : 0, c->stream));
    }
    if (c->profiling) { CK(cudaEventRecord(c->ev_th[1], c->stream)); c->prof_thermal = true; }
    if (hot_c_out) {
        CK(cudaMemcpyAsync(c->h_hot, c->td.hot, 3 * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
        CK(cudaStreamSynchronize(c->stream));
        memcpy(hot_c_out, c->h_hot, 3 * sizeof(float));
    }
    return HBF_OK;
}

int hbf_force_mode(hbf_ctx *c, int32_t mode, int64_t q_ppm) {
    if (!c || mode < 0 || mode > 3 || q_ppm < 1 || q_ppm > 1000000) return HBF_E_INVAL;
    DevState s;
    CK(cudaMemcpyAsync(&s, c->d_state, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    s.mode = mode; s.q_ppm = q_ppm;
    CK(cudaMemcpyAsync(c->d_state, &s, sizeof(s), cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (mode != HBF_MODE_SHUTDOWN) c->terminal = false;
    return HBF_OK;
}

int hbf_debug_wait_test(hbf_ctx *c, uint32_t poll_limit, uint32_t stage, uint32_t tile) {
    if (!c || stage > 2u) return HBF_E_INVAL;
    DevState s;
    CK(cudaMemcpyAsync(&s, c->d_state, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    c->spin_limit = poll_limit ? poll_limit : kSpinLimit; c->test_stage = stage; c->test_tile = tile;
    s.spin_limit = c->spin_limit; s.test_stage = stage; s.test_tile = tile;
    CK(cudaMemcpyAsync(c->d_state, &s, sizeof(s), cudaMemcpyHostToDevice, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_mode(hbf_ctx *c, int32_t *mode, int64_t *q_ppm) {
    if (!c) return HBF_E_INVAL;
    DevState s;
    CK(cudaMemcpyAsync(&s, c->d_state, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    if (mode) *mode = s.mode;
    if (q_ppm) *q_ppm = s.q_ppm;
    return HBF_OK;
}

int hbf_reset(hbf_ctx *c) {
    if (!c) return HBF_E_INVAL;
    DevState s; s.mode = HBF_MODE_NORMAL; s.poisoned = 0; s.q_ppm = 1000000;
    s.spin_limit = c->spin_limit; s.test_stage = c->test_stage; s.test_tile = c->test_tile; s.pad = 0;
    CK(cudaStreamSynchronize(c->stream));
    CK(cudaMemcpyAsync(c->d_state, &s, sizeof(s), cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemsetAsync(c->d_busy, 0, c->mp.n_queues * sizeof(int64_t), c->stream));
    CK(cudaMemsetAsync(c->d_pending, 0, c->mp.n_dies * sizeof(int64_t), c->stream));
    CK(cudaMemsetAsync(c->d_result, 0, sizeof(hbf_batch_result_t), c->stream));
    if (c->bin_ns) { CK(cudaMemsetAsync(c->d_ledger, 0, (size_t)c->n_bins * c->mp.n_dies * 8, c->stream)); c->cur_bin = 0; }
    if (c->d_bus_busy) CK(cudaMemsetAsync(c->d_bus_busy, 0, (size_t)c->mp.channels * 8, c->stream));
    if (c->ret_on) { int rc = retention_clear(c); if (rc != HBF_OK) return rc; }
    if (c->thermal) {
        const size_t nc = (size_t)c->td.H * c->td.W;
        CK(cudaMemsetAsync(c->td.theta[0], 0, nc * sizeof(float), c->stream));
        CK(cudaMemsetAsync(c->td.theta[1], 0, nc * sizeof(float), c->stream));
        CK(cudaMemsetAsync(c->td.comp, 0, nc * sizeof(float), c->stream));
        c->cur = 0;
    }
    CK(cudaStreamSynchronize(c->stream));
    c->terminal = false;
    return HBF_OK;
}

int hbf_get_busy_until(hbf_ctx *c, int64_t *host_out, uint64_t cap) {
    if (!c || !host_out || cap < c->mp.n_queues) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, c->d_busy, c->mp.n_queues * sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_pending_energy(hbf_ctx *c, int64_t *host_out, uint64_t cap) {
    if (!c || !host_out || cap < c->mp.n_dies) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, c->d_pending, c->mp.n_dies * sizeof(int64_t), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_get_temps(hbf_ctx *c, float *host_out, uint64_t cap) {
    if (!c || !c->thermal || !host_out) return HBF_E_INVAL;
    const size_t nc = (size_t)c->td.H * c->td.W;
    if (cap < nc) return HBF_E_INVAL;
    CK(cudaMemcpyAsync(host_out, c->td.theta[c->cur], nc * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    for (size_t i = 0; i < nc; ++i) host_out[i] += c->td.ambient_c;
    return HBF_OK;
}

int hbf_set_profiling(hbf_ctx *c, int on) {
    if (!c) return HBF_E_INVAL;
    if (on && !c->ev_made) {
        for (auto &e : c->ev) CK(cudaEventCreate(&e));
        for (auto &e : c->ev_th) CK(cudaEventCreate(&e));
        c->ev_made = true;
    }
    c->profiling = on != 0;
    if (!on) c->prof_submit = c->prof_thermal = false;
    return HBF_OK;
}

int hbf_get_profile(hbf_ctx *c, float *ms_out, uint32_t cap) {
    if (!c || !ms_out || cap < HBF_PROF_STAGES) return HBF_E_INVAL;
    for (int k = 0; k < HBF_PROF_STAGES; ++k) ms_out[k] = 0.0f;
    CK(cudaStreamSynchronize(c->stream));
    if (c->prof_submit) {
        for (int k = 1; k < 6; ++k) CK(cudaEventElapsedTime(&ms_out[k], c->ev[k], c->ev[k + 1]));
        if (c->prof_inorder) {                      // begin | in-order kernels | (second begin +) sort path ...
            CK(cudaEventElapsedTime(&ms_out[0], c->ev[0], c->ev[7]));
            CK(cudaEventElapsedTime(&ms_out[6], c->ev[7], c->ev[8]));
        } else {
            CK(cudaEventElapsedTime(&ms_out[0], c->ev[0], c->ev[1]));
        }
    }
    if (c->prof_thermal) CK(cudaEventElapsedTime(&ms_out[7], c->ev_th[0], c->ev_th[1]));
    return HBF_OK;
}

uint64_t hbf_kernel_launches(void) { return g_kernel_launches.load(); }

double hbf_euler_limit_ns(const hbf_ctx *c) { return c && c->thermal ? c->euler_limit_s * 1e9 : 0.0; }

// Sections of the blob after the header, in order: busy_until[queues], pending energy[dies], field and compensation
// [cells each]; then, for what is switched on: bus busy-until[channels]; ledger [n_bins][dies]; retention: the counters,
// per block damage (f64), disturb, PEC, epoch (u32 each), worn (u8), last plan position (u64), then the plan ring.
static size_t state_bytes(const hbf_ctx *c, size_t nc) {
    size_t need = sizeof(StateHeader) + (size_t)c->mp.n_queues * 8 + (size_t)c->mp.n_dies * 8 + nc * 8;
    if (c->d_bus_busy) need += (size_t)c->mp.channels * 8;
    if (c->bin_ns) need += (size_t)c->n_bins * c->mp.n_dies * 8;
    if (c->ret_on) need += sizeof(RetState) + (size_t)c->ret.n_blocks * (8 + 4 + 4 + 4 + 1 + 8) + (size_t)c->ret.plan_cap * 4;
    return need;
}

int hbf_get_state(hbf_ctx *c, void *host_buf, size_t *bytes) {
    if (!c || !bytes) return HBF_E_INVAL;
    const size_t nc = c->thermal ? (size_t)c->td.H * c->td.W : 0;
    const size_t need = state_bytes(c, nc);
    if (!host_buf) { *bytes = need; return HBF_OK; }
    if (*bytes < need) return HBF_E_INVAL;
    *bytes = need;
    char *p = static_cast<char *>(host_buf);
    DevState s;
    CK(cudaMemcpyAsync(&s, c->d_state, sizeof(s), cudaMemcpyDeviceToHost, c->stream));
    CK(cudaStreamSynchronize(c->stream));
    StateHeader h{};
    h.magic = kStateMagic; h.version = 2u; h.n_queues = c->mp.n_queues; h.n_dies = c->mp.n_dies; h.n_cells = (uint32_t)nc;
    h.mode = s.mode; h.q_ppm = s.q_ppm; h.poisoned = s.poisoned; h.cur = 0;
    h.flags = (c->d_bus_busy ? kStateBus : 0u) | (c->bin_ns ? kStateBins : 0u) | (c->ret_on ? kStateRetention : 0u);
    h.n_channels = c->mp.channels; h.bin_ns = c->bin_ns; h.cur_bin = c->cur_bin; h.n_bins = c->n_bins;
    h.ret_blocks = c->ret_on ? c->ret.n_blocks : 0; h.ret_plan_cap = c->ret_on ? c->ret.plan_cap : 0;
    memcpy(p, &h, sizeof(h)); p += sizeof(h);
    auto pull = [&](const void *dev, size_t n) { cudaError_t e = cudaMemcpyAsync(p, dev, n, cudaMemcpyDeviceToHost, c->stream); p += n; return e; };
    CK(pull(c->d_busy, (size_t)c->mp.n_queues * 8));
    CK(pull(c->d_pending, (size_t)c->mp.n_dies * 8));
    if (nc) { CK(pull(c->td.theta[c->cur], nc * 4)); CK(pull(c->td.comp, nc * 4)); }
    if (c->d_bus_busy) CK(pull(c->d_bus_busy, (size_t)c->mp.channels * 8));
    if (c->bin_ns) CK(pull(c->d_ledger, (size_t)c->n_bins * c->mp.n_dies * 8));
    if (c->ret_on) {
        const RetDev &r = c->ret;
        CK(pull(r.st, sizeof(RetState)));
        CK(pull(r.damage, r.n_blocks * 8)); CK(pull(r.disturb, r.n_blocks * 4)); CK(pull(r.pec, r.n_blocks * 4));
        CK(pull(r.epoch_of, r.n_blocks * 4)); CK(pull(r.worn, r.n_blocks)); CK(pull(r.last_pos, r.n_blocks * 8));
        CK(pull(r.plan, r.plan_cap * 4));
    }
    CK(cudaStreamSynchronize(c->stream));
    return HBF_OK;
}

int hbf_set_state(hbf_ctx *c, const void *host_buf, size_t bytes) {
    if (!c || !host_buf || bytes < sizeof(StateHeader)) return HBF_E_INVAL;
    const size_t nc = c->thermal ? (size_t)c->td.H * c->td.W : 0;
    const size_t need = state_bytes(c, nc);
    if (bytes < need) return HBF_E_INVAL;
    const char *p = static_cast<const char *>(host_buf);
    StateHeader h; memcpy(&h, p, sizeof(h)); p += sizeof(h);
    const uint32_t flags = (c->d_bus_busy ? kStateBus : 0u) | (c->bin_ns ? kStateBins : 0u) | (c->ret_on ? kStateRetention : 0u);
    if (h.magic != kStateMagic || h.version != 2u || h.n_queues != c->mp.n_queues || h.n_dies != c->mp.n_dies ||
        h.n_cells != (uint32_t)nc || h.mode < 0 || h.mode > 3 || h.q_ppm < 1 || h.q_ppm > 1000000) return HBF_E_INVAL;
    // the blob must come from a context with the same things switched on, at the same sizes
    if (h.flags != flags || h.n_channels != c->mp.channels || (c->bin_ns && (h.bin_ns != c->bin_ns || h.n_bins != c->n_bins)) ||
        (c->ret_on && (h.ret_blocks != c->ret.n_blocks || h.ret_plan_cap != c->ret.plan_cap))) return HBF_E_INVAL;
    DevState s; s.mode = h.mode; s.q_ppm = h.q_ppm; s.poisoned = h.poisoned;
    s.spin_limit = c->spin_limit; s.test_stage = c->test_stage; s.test_tile = c->test_tile; s.pad = 0;
    CK(cudaStreamSynchronize(c->stream));
    CK(cudaMemcpyAsync(c->d_state, &s, sizeof(s), cudaMemcpyHostToDevice, c->stream));
    auto push = [&](void *dev, size_t n) { cudaError_t e = cudaMemcpyAsync(dev, p, n, cudaMemcpyHostToDevice, c->stream); p += n; return e; };
    CK(push(c->d_busy, (size_t)c->mp.n_queues * 8));
    CK(push(c->d_pending, (size_t)c->mp.n_dies * 8));
    if (nc) { CK(push(c->td.theta[c->cur], nc * 4)); CK(push(c->td.comp, nc * 4)); }
    if (c->d_bus_busy) CK(push(c->d_bus_busy, (size_t)c->mp.channels * 8));
    if (c->bin_ns) { CK(push(c->d_ledger, (size_t)c->n_bins * c->mp.n_dies * 8)); c->cur_bin = h.cur_bin; }
    if (c->ret_on) {
        const RetDev &r = c->ret;
        CK(push(r.st, sizeof(RetState)));
        CK(push(r.damage, r.n_blocks * 8)); CK(push(r.disturb, r.n_blocks * 4)); CK(push(r.pec, r.n_blocks * 4));
        CK(push(r.epoch_of, r.n_blocks * 4)); CK(push(r.worn, r.n_blocks)); CK(push(r.last_pos, r.n_blocks * 8));
        CK(push(r.plan, r.plan_cap * 4));
    }
    CK(cudaStreamSynchronize(c->stream));
    c->terminal = (h.mode == HBF_MODE_SHUTDOWN) ? c->terminal : false;
    return HBF_OK;
}

}  // extern "C"
