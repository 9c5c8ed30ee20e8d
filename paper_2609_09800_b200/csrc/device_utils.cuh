// Small device helpers: memory-model loads/stores for look-back words, warp reductions, and the
// per-access arithmetic (classification, decode, service terms) used by every path.
#pragma once
#include "hbf_dev.cuh"

namespace hbf {

__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p) {
    uint32_t v; asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void st_relaxed_u32(uint32_t *p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t *p) {
    uint32_t v; asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t *p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ int64_t ld_relaxed_s64(const int64_t *p) {
    int64_t v; asm volatile("ld.relaxed.gpu.global.s64 %0, [%1];" : "=l"(v) : "l"(p) : "memory"); return v;
}
__device__ __forceinline__ void st_relaxed_s64(int64_t *p, int64_t v) {
    asm volatile("st.relaxed.gpu.global.s64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint64_t ld_nc_u64(const uint64_t *p) {
    uint64_t v; asm volatile("ld.global.nc.u64 %0, [%1];" : "=l"(v) : "l"(p)); return v;
}

// ---- division by a run-time constant ----------------------------------------------------------------
// For d not a power of two, l = ceil(log2 d), magic = floor(2^(63+l) / d) + 1: floor(n / d) =
// mulhi(n, magic) >> (l - 1) for every n < 2^63 (the error term n * (magic*d - 2^(63+l)) stays below 2^(63+l)).
__host__ __device__ inline Div64 make_div64(uint64_t d) {
    Div64 r; r.magic = 0; r.shift = 0; r.pow2 = 0;
    if ((d & (d - 1)) == 0) { r.pow2 = 1; while ((1ull << r.shift) < d) ++r.shift; return r; }
    uint32_t l = 0; while (l < 64 && (1ull << l) < d) ++l;
    const unsigned __int128 num = (unsigned __int128)1 << (63 + l);
    r.magic = (uint64_t)(num / d) + 1ull; r.shift = l - 1;
    return r;
}
__device__ __forceinline__ uint64_t div64(uint64_t n, const Div64 &d) {
    return d.pow2 ? (n >> d.shift) : (__umul64hi(n, d.magic) >> d.shift);
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }
__device__ __forceinline__ unsigned lanemask_lt() { unsigned m; asm("mov.u32 %0, %%lanemask_lt;" : "=r"(m)); return m; }

__device__ __forceinline__ long long warp_sum(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ long long warp_max(long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { long long w = __shfl_xor_sync(0xffffffffu, v, o); v = w > v ? w : v; }
    return v;
}
__device__ __forceinline__ unsigned long long warp_or(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v |= __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_and(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v &= __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- classification (Design D1) ---------------------------------------------------------------

// Ranges are sorted by base and disjoint.  Returns the status; *g receives the range index.
__device__ __forceinline__ int classify(const RangeSnap &rs, uint64_t addr, int64_t issue, uint32_t bytes,
                                        uint32_t flags, int *g) {
    if (bytes == 0u || (flags & ~1u) != 0u || issue < 0 || issue >= HBF_ISSUE_LIMIT) return HBF_ST_UNSUPPORTED;
    int k;
    if (rs.count == 1u) {                        // the common registration: one range
        k = addr >= rs.base[0] ? 0 : -1;
    } else {
        int lo = 0, hi = (int)rs.count;          // last range with base <= addr
        while (lo < hi) { int mid = (lo + hi) >> 1; if (rs.base[mid] <= addr) lo = mid + 1; else hi = mid; }
        k = lo - 1;
    }
    if (k < 0) return HBF_ST_NATIVE;
    uint64_t rel = addr - rs.base[k];
    if (rel >= rs.length[k]) return HBF_ST_NATIVE;
    *g = k;
    if ((uint64_t)bytes > rs.length[k] - rel) return HBF_ST_FAULT_PARTIAL;
    uint32_t need = (flags & 1u) ? (uint32_t)HBF_PERM_PROGRAM : (uint32_t)HBF_PERM_READ;
    if (!(rs.perms[k] & need)) return HBF_ST_FAULT_PERM;
    return HBF_ST_READY;
}

// ---- decode ---------------------------------------------------------------------------------------

struct Decoded { uint32_t queue, die; uint32_t npages; };

__device__ __forceinline__ Decoded decode(const ModelParams &mp, uint64_t off, uint32_t bytes) {
    Decoded d;
    uint64_t u = off >> mp.stripe_shift;
    uint32_t ch, di, pl;
    if (mp.pow2_geom) {
        ch = (uint32_t)u & (mp.channels - 1u);
        di = (uint32_t)(u >> mp.ch_shift) & (mp.dies - 1u);
        pl = (uint32_t)(u >> (mp.ch_shift + mp.die_shift)) & (mp.planes - 1u);
    } else {
        ch = (uint32_t)(u % mp.channels);
        uint64_t v = u / mp.channels;
        di = (uint32_t)(v % mp.dies);
        pl = (uint32_t)((v / mp.dies) % mp.planes);
    }
    d.die = ch * mp.dies + di;
    d.queue = mp.queue_level == 0u ? d.die * mp.planes + pl : d.die;
    uint64_t in_page = off & ((1ull << mp.page_shift) - 1ull);
    d.npages = (uint32_t)((in_page + bytes + (1ull << mp.page_shift) - 1ull) >> mp.page_shift);
    return d;
}

// ---- retention: block (erase unit) that holds a media offset's page: ((channel, die, plane) * blocks_per_plane + block)
__device__ __forceinline__ uint64_t ret_block_of(const ModelParams &mp, const RetDev &r, uint64_t off) {
    const uint64_t u = off >> mp.stripe_shift;
    uint32_t ch, di, pl; uint64_t row;
    if (mp.pow2_geom) {
        ch = (uint32_t)u & (mp.channels - 1u);
        di = (uint32_t)(u >> mp.ch_shift) & (mp.dies - 1u);
        pl = (uint32_t)(u >> (mp.ch_shift + mp.die_shift)) & (mp.planes - 1u);
        row = u >> (mp.ch_shift + mp.die_shift + mp.plane_shift);
    } else {
        ch = (uint32_t)(u % mp.channels);
        uint64_t v = u / mp.channels;
        di = (uint32_t)(v % mp.dies); v /= mp.dies;
        pl = (uint32_t)(v % mp.planes); row = v / mp.planes;
    }
    const uint64_t in_stripe = (off & ((1ull << mp.stripe_shift) - 1ull)) >> mp.page_shift;
    const uint64_t page = (row << mp.pages_per_stripe_shift) + in_stripe;
    const uint64_t blk = div64(page, r.div_ppb);             // page < 2^63 always
    const uint64_t bip = blk - div64(blk, r.div_bpp) * r.bpp;
    return (((uint64_t)ch * mp.dies + di) * mp.planes + pl) * r.bpp + bip;
}

// ---- service terms (Eq. 3 for the array time; transfer is pure latency) ---------------------------

struct Terms { int64_t s, xfer, energy, cb; };

__device__ __forceinline__ Terms service_terms(const ModelParams &mp, uint32_t bytes, uint32_t npages, uint32_t op,
                                               int64_t q_ppm, const Div64 &div_q) {
    Terms t;
    uint32_t gs = op ? mp.prog_gran_shift : mp.read_gran_shift;
    uint64_t cb = (((uint64_t)bytes + (1ull << gs) - 1ull) >> gs) << gs;
    t.cb = (int64_t)cb;
    t.xfer = (int64_t)div64(cb * 1000ull + mp.chan_bytes_per_us - 1ull, mp.div_chan);
    int64_t s0 = (int64_t)npages * (op ? mp.t_prog_ns : mp.t_read_ns);
    t.s = q_ppm == 1000000 ? s0 : (int64_t)div64((uint64_t)s0 * 1000000ull + (uint64_t)q_ppm - 1ull, div_q);
    t.energy = op ? mp.e_cmd_prog_pj + mp.e_byte_prog_pj * (int64_t)cb : mp.e_cmd_read_pj + mp.e_byte_read_pj * (int64_t)cb;
    return t;
}

}  // namespace hbf
