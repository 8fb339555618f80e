// Fault-injected mixed-precision GEMM for sm_100a.
//
// One persistent CTA per SM walks 128 x BN output tiles. Warp roles:
//   warp 0    TMA producer: k-tiles of A (128 rows x 128 bytes) and Bt (BN rows x 128 bytes)
//             into a ring of 128-byte-swizzled shared-memory stages
//   warp 1    MMA issuer: tcgen05.mma into one of two TMEM accumulators; flips operand
//             sites in the staged tiles before the tensor core reads them; pauses at the
//             k-step boundaries where an accumulator or product-term site takes effect
//   warp 2    TMEM allocation / release
//   warps 4-7 epilogue: TMEM -> registers, accumulator / term write-back sites at the
//             paused boundaries, output-site flips, BoundCheck flags (+ correction), stores
//
// The fault-site table is decoded once per CTA into a list of the entries that touch any of
// its tiles; a CTA whose list is empty never looks at a site again.
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "checks.cuh"
#include "gemm_sm100.cuh"
#include "ptx_sm100.cuh"

namespace mpg {

namespace {

constexpr uint32_t NONE = 0xFFFFFFFFu;
constexpr int BM = 128;
constexpr int NUM_THREADS = 256;
constexpr int MAX_STAGES = 8;

template <int BN>
struct Cfg {
    static constexpr int A_BYTES = BM * 128;
    static constexpr int B_BYTES = BN * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (200 * 1024 / STAGE_BYTES) < MAX_STAGES ? (200 * 1024 / STAGE_BYTES) : MAX_STAGES;
    static constexpr int TMEM_COLS = 2 * BN;   // two accumulators; 128, 256 or 512 columns
    static_assert(BN == 64 || BN == 128 || BN == 256, "BN must be 64, 128 or 256");
};

// Control block that follows the stages in dynamic shared memory.
struct alignas(16) Control {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t pause_full;
    uint64_t pause_done;
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t site_count;
    uint32_t pad;
    uint32_t scan[NUM_THREADS];
    uint16_t site_idx[MPGEMMFI_MAX_FAULTS];
};

struct TileCtx {
    const GemmParams *p;
    const Control *ctl;
    uint32_t m0, n0;
    int bn;
};

__device__ __forceinline__ bool in_tile_rows(const TileCtx &c, uint32_t row) { return row - c.m0 < (uint32_t)BM; }
__device__ __forceinline__ bool in_tile_cols(const TileCtx &c, uint32_t col) { return col - c.n0 < (uint32_t)c.bn; }

// smallest k-tile >= kt_from in which this tile has an operand site (warp-wide)
__device__ uint32_t scan_next_operand(const TileCtx &c, uint32_t kt_from, int lane)
{
    const uint32_t ks = (uint32_t)kstep_of(c.p->dtype);
    uint32_t best = NONE;
    for (uint32_t i = lane; i < c.ctl->site_count; i += 32) {
        const mpgemmfi_site s = load_site(c.p->sites, c.ctl->site_idx[i]);
        const bool hit = (s.kind == MPGEMMFI_SITE_A && in_tile_rows(c, s.row)) ||
                         (s.kind == MPGEMMFI_SITE_B && in_tile_cols(c, s.col));
        if (hit && s.k / ks >= kt_from) best = min(best, s.k / ks);
    }
    return __reduce_min_sync(0xFFFFFFFFu, best);
}

// smallest boundary >= b_from at which this tile has an accumulator / term site (warp-wide)
__device__ uint32_t scan_next_boundary(const TileCtx &c, uint32_t b_from, int lane)
{
    uint32_t best = NONE;
    for (uint32_t i = lane; i < c.ctl->site_count; i += 32) {
        const mpgemmfi_site s = load_site(c.p->sites, c.ctl->site_idx[i]);
        if ((s.kind == MPGEMMFI_SITE_ACC || s.kind == MPGEMMFI_SITE_TERM) && in_tile_rows(c, s.row) &&
            in_tile_cols(c, s.col)) {
            const uint32_t b = site_boundary(s, c.p->dtype, c.p->K);
            if (b >= b_from) best = min(best, b);
        }
    }
    return __reduce_min_sync(0xFFFFFFFFu, best);
}

__device__ bool scan_has_out(const TileCtx &c, int lane)
{
    bool any = false;
    for (uint32_t i = lane; i < c.ctl->site_count; i += 32) {
        const mpgemmfi_site s = load_site(c.p->sites, c.ctl->site_idx[i]);
        any |= s.kind == MPGEMMFI_SITE_OUT && in_tile_rows(c, s.row) && in_tile_cols(c, s.col);
    }
    return __any_sync(0xFFFFFFFFu, any);
}

__device__ __forceinline__ mpgemmfi_site_log *site_log(const GemmParams &p, uint32_t idx)
{
    return p.flags ? reinterpret_cast<mpgemmfi_site_log *>(p.flags + MPGEMMFI_HEADER_WORDS) + idx : nullptr;
}

__device__ __forceinline__ void write_log(const GemmParams &p, uint32_t idx, uint32_t before, uint32_t after,
                                          uint32_t fin, uint32_t status)
{
    mpgemmfi_site_log *l = site_log(p, idx);
    if (l) { l->before_bits = before; l->after_bits = after; l->final_bits = fin; l->status = status; }
}

// byte offset of element (row r, byte kb of the 128-byte row) inside a 128-byte-swizzled tile
__device__ __forceinline__ uint32_t swizzled_offset(uint32_t r, uint32_t kb)
{
    return r * 128u + ((((kb >> 4) ^ (r & 7u)) << 4) | (kb & 15u));
}

// One thread: XOR the operand sites of k-tile `kt` into the staged A / Bt tiles, table order.
__device__ void apply_operand_sites(const TileCtx &c, uint32_t kt, uint8_t *smem_a, uint8_t *smem_b)
{
    const GemmParams &p = *c.p;
    const uint32_t ks = (uint32_t)kstep_of(p.dtype);
    const uint32_t es = (uint32_t)esize_of(p.dtype);
    for (uint32_t i = 0; i < c.ctl->site_count; ++i) {
        const uint32_t idx = c.ctl->site_idx[i];
        const mpgemmfi_site s = load_site(p.sites, idx);
        uint8_t *tile;
        uint32_t r;
        bool log_here;
        if (s.kind == MPGEMMFI_SITE_A && in_tile_rows(c, s.row)) { tile = smem_a; r = s.row - c.m0; log_here = c.n0 == 0; }
        else if (s.kind == MPGEMMFI_SITE_B && in_tile_cols(c, s.col)) { tile = smem_b; r = s.col - c.n0; log_here = c.m0 == 0; }
        else continue;
        if (s.k / ks != kt) continue;
        uint8_t *ptr = tile + swizzled_offset(r, (s.k % ks) * es);
        uint32_t before, after;
        if (es == 2) {
            unsigned short *w = reinterpret_cast<unsigned short *>(ptr);
            before = *w;
            after = flip_operand(p.dtype, before, s.xor_mask);
            *w = (unsigned short)after;
        } else {
            uint32_t *w = reinterpret_cast<uint32_t *>(ptr);
            before = *w & 0xFFFFE000u;
            after = flip_operand(p.dtype, before, s.xor_mask);
            *w = after;
        }
        if (log_here) write_log(p, idx, before, after, after, 1u);
    }
}

// operand word of A[row,k] or Bt[col,k] with every operand site of the table applied
__device__ uint32_t faulty_operand(const TileCtx &c, bool is_a, uint32_t rc, uint32_t k)
{
    const GemmParams &p = *c.p;
    uint32_t w = load_operand(p.dtype, is_a ? p.A : p.Bt, (size_t)rc * p.K + k);
    for (uint32_t i = 0; i < c.ctl->site_count; ++i) {
        const mpgemmfi_site s = load_site(p.sites, c.ctl->site_idx[i]);
        if (s.k != k) continue;
        if (is_a ? (s.kind == MPGEMMFI_SITE_A && s.row == rc) : (s.kind == MPGEMMFI_SITE_B && s.col == rc))
            w = flip_operand(p.dtype, w, s.xor_mask);
    }
    return w;
}

// Epilogue warp of lane quarter q: apply, in table order, the accumulator and term sites of
// boundary b that live in its 32 TMEM lanes.
__device__ void apply_boundary_sites(const TileCtx &c, uint32_t b, uint32_t tmem_acc, int q, int lane)
{
    const GemmParams &p = *c.p;
    for (uint32_t i = 0; i < c.ctl->site_count; ++i) {
        const uint32_t idx = c.ctl->site_idx[i];
        const mpgemmfi_site s = load_site(p.sites, idx);
        if (!(s.kind == MPGEMMFI_SITE_ACC || s.kind == MPGEMMFI_SITE_TERM)) continue;
        if (!in_tile_rows(c, s.row) || !in_tile_cols(c, s.col)) continue;
        if (site_boundary(s, p.dtype, p.K) != b) continue;
        const uint32_t r = s.row - c.m0;
        if ((int)(r >> 5) != q) continue;
        const uint32_t taddr = tmem_acc + ((uint32_t)(q * 32) << 16) + (s.col - c.n0);
        uint32_t v = tmem_ld_1(taddr);
        tmem_wait_ld();
        if (lane == (int)(r & 31u)) {
            if (s.kind == MPGEMMFI_SITE_ACC) {
                const uint32_t before = v;
                v ^= s.xor_mask;
                write_log(p, idx, before, v, v, 1u);
            } else {
                // write-back of Eq. 1-2: remove the clean product, add the faulty (checked) one
                const uint32_t aw = faulty_operand(c, true, s.row, s.k);
                const uint32_t bw = faulty_operand(c, false, s.col, s.k);
                const float a = widen_operand(p.dtype, aw), bb = widen_operand(p.dtype, bw);
                const float re2 = __fmul_rn(a, bb);
                const uint32_t before = f32_bits(re2);
                const uint32_t after = before ^ s.xor_mask;
                bool det;
                const uint32_t fin = product_check(p.detect_mode, after, f32_bits(a), f32_bits(bb), det);
                const float rep = __fsub_rn(bits_f32(v), re2);
                v = f32_bits(__fadd_rn(rep, bits_f32(fin)));
                write_log(p, idx, before, after, fin, 1u | (det ? 4u : 0u));
            }
        }
        tmem_st_1(taddr, v);
        tmem_wait_st();
    }
}

// Output sites of one thread's row inside the 32-column chunk starting at column c0.
// pass 0: XOR and log before/after; pass 1 (after the check): log the final bits.
__device__ void apply_out_sites(const TileCtx &c, uint32_t row, uint32_t c0, uint32_t (&v)[32], int pass)
{
    const GemmParams &p = *c.p;
    for (uint32_t i = 0; i < c.ctl->site_count; ++i) {
        const uint32_t idx = c.ctl->site_idx[i];
        const mpgemmfi_site s = load_site(p.sites, idx);
        if (s.kind != MPGEMMFI_SITE_OUT || s.row != row || s.col - c0 >= 32u) continue;
        const uint32_t j = s.col - c0;
#pragma unroll
        for (uint32_t jj = 0; jj < 32; ++jj) {
            if (jj == j) {
                if (pass == 0) {
                    const uint32_t before = v[jj];
                    v[jj] ^= s.xor_mask;
                    write_log(p, idx, before, v[jj], v[jj], 1u);
                } else {
                    mpgemmfi_site_log *l = site_log(p, idx);
                    if (l) l->final_bits = v[jj];
                }
            }
        }
    }
}

template <int BN>
__device__ bool site_touches_cta(const mpgemmfi_site &s, const GemmParams &p)
{
    const uint32_t g = gridDim.x, bid = blockIdx.x;
    if (s.kind == MPGEMMFI_SITE_A) {
        const uint32_t tm = s.row / BM;
        for (uint32_t tn = 0; tn < (uint32_t)p.tiles_n; ++tn)
            if ((tn * p.tiles_m + tm) % g == bid) return true;
        return false;
    }
    if (s.kind == MPGEMMFI_SITE_B) {
        const uint32_t tn = s.col / BN;
        for (uint32_t tm = 0; tm < (uint32_t)p.tiles_m; ++tm)
            if ((tn * p.tiles_m + tm) % g == bid) return true;
        return false;
    }
    return ((s.col / BN) * p.tiles_m + s.row / BM) % g == bid;
}

// All threads: ordered list of the valid sites that touch a tile of this CTA. CTA 0 also
// reports invalid entries (skipped) and the applied count.
template <int BN>
__device__ void build_site_list(const GemmParams &p, Control *ctl)
{
    const int tid = threadIdx.x;
    const int n = p.n_faults;
    if (n == 0) {
        if (tid == 0) ctl->site_count = 0;
        return;
    }
    const int per = (n + NUM_THREADS - 1) / NUM_THREADS;
    const int beg = min(n, tid * per), end = min(n, beg + per);
    uint32_t cnt = 0, n_valid = 0, n_bad = 0;
    for (int i = beg; i < end; ++i) {
        const mpgemmfi_site s = load_site(p.sites, i);
        const bool ok = site_valid(s, p.dtype, p.M, p.N, p.K);
        if (ok) { n_valid++; cnt += site_touches_cta<BN>(s, p) ? 1u : 0u; }
        else {
            n_bad++;
            if (blockIdx.x == 0) write_log(p, i, 0u, 0u, 0u, 2u);
        }
    }
    if (blockIdx.x == 0 && p.flags) {
        if (n_valid) atomicAdd(&p.flags[3], n_valid);
        if (n_bad) { atomicAdd(&p.flags[4], n_bad); atomicOr(&p.flags[0], MPGEMMFI_STATUS_SITE_SKIPPED); }
    }
    ctl->scan[tid] = cnt;
    __syncthreads();
    if (tid == 0) {
        uint32_t run = 0;
        for (int t = 0; t < NUM_THREADS; ++t) { const uint32_t x = ctl->scan[t]; ctl->scan[t] = run; run += x; }
        ctl->site_count = run;
    }
    __syncthreads();
    uint32_t off = ctl->scan[tid];
    for (int i = beg; i < end; ++i) {
        const mpgemmfi_site s = load_site(p.sites, i);
        if (site_valid(s, p.dtype, p.M, p.N, p.K) && site_touches_cta<BN>(s, p)) ctl->site_idx[off++] = (uint16_t)i;
    }
}

template <int BN, bool kTF32>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, const GemmParams p)
{
    using C = Cfg<BN>;
    constexpr int KT = kTF32 ? 32 : 64;      // elements per 128-byte row
    constexpr int STAGES = C::STAGES;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Control *ctl = reinterpret_cast<Control *>(smem + STAGES * C::STAGE_BYTES);
    volatile uint32_t *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t num_kt = (uint32_t)p.num_kt;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&ctl->full[s]), 1); mbar_init(smem_u32(&ctl->empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->acc_full[s]), 1); mbar_init(smem_u32(&ctl->acc_empty[s]), 4); }
        mbar_init(smem_u32(&ctl->pause_full), 1);
        mbar_init(smem_u32(&ctl->pause_done), 4);
        ctl->abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
    }
    if (warp == 2) {
        tmem_alloc(smem_u32(&ctl->tmem_base), C::TMEM_COLS);
        tmem_relinquish();
    }
    build_site_list<BN>(p, ctl);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();

    const uint32_t tmem_base = ctl->tmem_base;
    const bool has_sites = ctl->site_count != 0;
    TileCtx tc;
    tc.p = &p; tc.ctl = ctl; tc.bn = BN;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t stage = 0, phase = 0, armed = 0, armed_parity = 0;
            bool ok = true;
            for (uint32_t t = blockIdx.x; ok && t < (uint32_t)p.num_tiles; t += gridDim.x) {
                const int m0 = (int)(t % p.tiles_m) * BM, n0 = (int)(t / p.tiles_m) * BN;
                for (uint32_t kt = 0; kt < num_kt; ++kt) {
                    if (!mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&ctl->full[stage]);
                    uint8_t *sa = smem + stage * C::STAGE_BYTES;
                    mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                    tma_load_2d(smem_u32(sa), &tm_a, bar, (int)(kt * KT), m0);
                    tma_load_2d(smem_u32(sa + C::A_BYTES), &tm_b, bar, (int)(kt * KT), n0);
                    armed |= 1u << stage;
                    armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
            // wait (bounded) until every copy this thread started has landed
            uint32_t never = 0;
            for (int s = 0; s < STAGES; ++s)
                if (armed & (1u << s))
                    mbar_wait(smem_u32(&ctl->full[s]), (armed_parity >> s) & 1u, &never, 1000000000ull);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_instr_desc((uint32_t)p.dtype, BM, BN);
        uint32_t stage = 0, phase = 0, lt = 0, pause_phase = 0;
        bool ok = true;
        for (uint32_t t = blockIdx.x; ok && t < (uint32_t)p.num_tiles; t += gridDim.x, ++lt) {
            const uint32_t as = lt & 1u, ap = (lt >> 1) & 1u;
            tc.m0 = (t % p.tiles_m) * BM; tc.n0 = (t / p.tiles_m) * BN;
            uint32_t next_op = NONE, next_b = NONE;
            if (has_sites) { next_op = scan_next_operand(tc, 0, lane); next_b = scan_next_boundary(tc, 1, lane); }
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->acc_empty[as]), ap ^ 1u, abort_flag));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + as * BN;
            for (uint32_t kt = 0; kt < num_kt; ++kt) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                uint8_t *sa = smem + stage * C::STAGE_BYTES;
                if (kt == next_op) {
                    if (lane == 0) {
                        apply_operand_sites(tc, kt, sa, sa + C::A_BYTES);
                        fence_proxy_async_smem();
                    }
                    __syncwarp();
                    next_op = scan_next_operand(tc, kt + 1, lane);
                }
                if (lane == 0) {
                    const uint64_t a_desc = umma_smem_desc_sw128(smem_u32(sa));
                    const uint64_t b_desc = umma_smem_desc_sw128(smem_u32(sa + C::A_BYTES));
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k)     // 4 x 32 bytes along K inside the swizzle row
                        umma_ss<kTF32>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kt | k) != 0 ? 1u : 0u);
                    umma_commit(smem_u32(&ctl->empty[stage]));
                }
                __syncwarp();
                if (kt + 1 == next_b) {
                    // an accumulator / term site takes effect here: let the epilogue warps edit TMEM
                    if (lane == 0) umma_commit(smem_u32(&ctl->pause_full));
                    __syncwarp();
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->pause_done), pause_phase, abort_flag));
                    if (!ok) break;
                    pause_phase ^= 1u;
                    tc_fence_after_sync();
                    next_b = scan_next_boundary(tc, kt + 2, lane);
                }
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
            if (!ok) break;
            if (lane == 0) umma_commit(smem_u32(&ctl->acc_full[as]));
            __syncwarp();
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;
        const bool do_bound = (p.detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK) == MPGEMMFI_DETECT_BOUNDCHECK;
        const bool do_corr = do_bound && (p.detect_mode & MPGEMMFI_CORRECT);
        uint32_t lt = 0, pause_phase = 0, n_det = 0;
        uint32_t *bitmap = p.flags ? p.flags + MPGEMMFI_HEADER_WORDS + 4 * (size_t)p.n_faults : nullptr;
        bool ok = true;
        for (uint32_t t = blockIdx.x; ok && t < (uint32_t)p.num_tiles; t += gridDim.x, ++lt) {
            const uint32_t as = lt & 1u, ap = (lt >> 1) & 1u;
            tc.m0 = (t % p.tiles_m) * BM; tc.n0 = (t / p.tiles_m) * BN;
            const uint32_t tmem_acc = tmem_base + as * BN;
            bool tile_has_out = false;
            if (has_sites) {
                uint32_t b = scan_next_boundary(tc, 1, lane);
                while (b != NONE) {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->pause_full), pause_phase, abort_flag));
                    if (!ok) break;
                    pause_phase ^= 1u;
                    tc_fence_after_sync();
                    apply_boundary_sites(tc, b, tmem_acc, q, lane);
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->pause_done));
                    b = scan_next_boundary(tc, b + 1, lane);
                }
                if (!ok) break;
                tile_has_out = scan_has_out(tc, lane);
            }
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->acc_full[as]), ap, abort_flag));
            if (!ok) break;
            tc_fence_after_sync();

            const uint32_t row = tc.m0 + (uint32_t)(q * 32 + lane);
            const bool row_ok = row < (uint32_t)p.M;
            float *crow = p.C + (size_t)row * p.N;
            uint32_t flagw[BN / 32];
#pragma unroll
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
                tmem_wait_ld();
                if (c == BN / 32 - 1) {
                    // accumulator fully read: hand the TMEM buffer back to the MMA warp
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&ctl->acc_empty[as]));
                }
                const uint32_t c0 = tc.n0 + (uint32_t)(c * 32);
                if (tile_has_out && row_ok) apply_out_sites(tc, row, c0, v, 0);
                uint32_t fw = 0;
                if (do_bound) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const bool det = boundcheck_detect(v[j]);
                        fw |= (det ? 1u : 0u) << j;
                        if (do_corr && det) v[j] = boundcheck_clear(v[j]);
                    }
                    // columns past N hold zeros (zero-filled operand rows) and never flag
                }
                if (tile_has_out && row_ok) apply_out_sites(tc, row, c0, v, 1);
                flagw[c] = fw;
                if (row_ok) {
                    if (c0 + 32 <= (uint32_t)p.N && p.c_vec_ok) {
                        float4 *dst = reinterpret_cast<float4 *>(crow + c0);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            dst[j] = make_float4(bits_f32(v[4 * j]), bits_f32(v[4 * j + 1]), bits_f32(v[4 * j + 2]),
                                                 bits_f32(v[4 * j + 3]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < (uint32_t)p.N) crow[c0 + j] = bits_f32(v[j]);
                    }
                }
            }
            if (bitmap && row_ok) {
                uint32_t *frow = bitmap + (size_t)row * p.wpr + tc.n0 / 32;
#pragma unroll
                for (int c = 0; c < BN / 32; ++c) {
                    if (tc.n0 / 32 + c < (uint32_t)p.wpr) frow[c] = flagw[c];
                    n_det += __popc(flagw[c]);
                }
            }
        }
        n_det = __reduce_add_sync(0xFFFFFFFFu, n_det);
        if (lane == 0 && n_det && p.flags) {
            atomicAdd(&p.flags[1], n_det);
            if (do_corr) atomicAdd(&p.flags[2], n_det);
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem_base, C::TMEM_COLS);
    if (threadIdx.x == 0 && ctl->abort_flag && p.flags) atomicOr(&p.flags[0], MPGEMMFI_STATUS_WAIT_LIMIT);
}

template <int BN, bool kTF32>
cudaError_t launch_one(const CUtensorMap &tm_a, const CUtensorMap &tm_b, const GemmParams &p, int grid,
                       cudaStream_t stream)
{
    using C = Cfg<BN>;
    const size_t smem = (size_t)C::STAGES * C::STAGE_BYTES + sizeof(Control) + 1024;
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(gemm_kernel<BN, kTF32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    gemm_kernel<BN, kTF32><<<grid, NUM_THREADS, smem, stream>>>(tm_a, tm_b, p);
    return cudaGetLastError();
}

}  // namespace

int gemm_stage_count(int bn)
{
    return bn == 256 ? Cfg<256>::STAGES : (bn == 128 ? Cfg<128>::STAGES : Cfg<64>::STAGES);
}

cudaError_t launch_gemm(int bn, const CUtensorMap &tm_a, const CUtensorMap &tm_b, const GemmParams &p, int grid,
                        cudaStream_t stream)
{
    const bool tf32 = p.dtype == MPGEMMFI_TF32;
    switch (bn) {
    case 256: return tf32 ? launch_one<256, true>(tm_a, tm_b, p, grid, stream) : launch_one<256, false>(tm_a, tm_b, p, grid, stream);
    case 128: return tf32 ? launch_one<128, true>(tm_a, tm_b, p, grid, stream) : launch_one<128, false>(tm_a, tm_b, p, grid, stream);
    default:  return tf32 ? launch_one<64, true>(tm_a, tm_b, p, grid, stream) : launch_one<64, false>(tm_a, tm_b, p, grid, stream);
    }
}

}  // namespace mpg
