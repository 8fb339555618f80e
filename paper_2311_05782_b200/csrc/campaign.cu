// Injection campaign: per-trial evaluation kernels that run after ONE clean GEMM.
//
// Every trial is one fault site applied alone. Only the output elements the site can reach
// are evaluated:
//   OUT        flip the clean element
//   ACC, TERM  redo the element's dot product in k order on the FP32 ALUs, once clean and
//              once with the site active (the clean pass is the trial's reference)
//   A, B       c' = (c - a*b) + a'*b for every element of the affected row / column
//              (the write-back of Eq. 1-2 applied to a finished sum)
// and every evaluated element goes through the output check.
//
//   B (long columns, short rows): batched by row panel, see panel_kernel
//
// Scratch (the "schedule"): three compacted lists of trial indices (A sites, B sites,
// single-element sites) plus their counters, so that each evaluation kernel walks only its
// own kind of trial.
#include <cstdint>
#include <cuda_runtime.h>

#include "campaign.cuh"
#include "checks.cuh"

namespace mpg {

namespace {

constexpr unsigned long long HASH_MUL = 0x9E3779B97F4A7C15ull;
constexpr int VEC_THREADS = 256;

struct Stats {
    uint32_t n_det;
    uint32_t first;
    uint32_t maxdev_bits;   // non-negative floats order like their bit patterns
    uint32_t changed;
    unsigned long long hash;
};

__device__ __forceinline__ void stats_init(Stats &s)
{
    s.n_det = 0; s.first = 0xFFFFFFFFu; s.maxdev_bits = 0; s.changed = 0; s.hash = 0ull;
}

// run the output check on one evaluated element and fold it into the trial's statistics
__device__ __forceinline__ uint32_t stats_account(Stats &s, int detect_mode, uint32_t value_bits, uint32_t clean_bits,
                                                  uint32_t lin)
{
    bool det;
    const uint32_t fin = output_check(detect_mode, value_bits, det);
    if (det) {
        s.n_det++;
        s.hash += ((unsigned long long)lin + 1ull) * HASH_MUL;
        s.first = min(s.first, lin);
    }
    if (fin != clean_bits) s.changed = 1;
    float dev = fabsf(__fsub_rn(bits_f32(fin), bits_f32(clean_bits)));
    if (dev != dev) dev = __uint_as_float(0x7F800000u);      // NaN deviation counts as +inf
    s.maxdev_bits = max(s.maxdev_bits, f32_bits(dev));
    return fin;
}

__device__ __forceinline__ void stats_warp_reduce(Stats &s)
{
    s.n_det = __reduce_add_sync(0xFFFFFFFFu, s.n_det);
    s.first = __reduce_min_sync(0xFFFFFFFFu, s.first);
    s.maxdev_bits = __reduce_max_sync(0xFFFFFFFFu, s.maxdev_bits);
    s.changed = __reduce_or_sync(0xFFFFFFFFu, s.changed);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s.hash += __shfl_xor_sync(0xFFFFFFFFu, s.hash, o);
}

__device__ __forceinline__ uint32_t status_bits(const Stats &s, int detect_mode)
{
    const bool corr = (detect_mode & MPGEMMFI_CORRECT) &&
                      (detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK) == MPGEMMFI_DETECT_BOUNDCHECK;
    return (s.changed ? 1u : 0u) | (s.n_det ? 2u : 0u) | ((s.n_det && corr) ? 4u : 0u);
}

// ---------------------------------------------------------------- schedule

__global__ void schedule_kernel(CampaignParams p)
{
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= p.n_trials) return;
    const mpgemmfi_site s = load_site(p.sites, t);
    mpgemmfi_trial_record r;
    r.status = 0; r.kind = s.kind; r.primary_index = 0; r.before_bits = 0; r.after_bits = 0; r.final_bits = 0;
    r.n_affected = 0; r.n_detected = 0; r.idx_hash = 0ull; r.first_detected = 0xFFFFFFFFu; r.max_abs_dev = 0.0f;
    if (!site_valid(s, p.dtype, p.M, p.N, p.K)) {
        r.status = 1u << 8;
    } else if (s.kind == MPGEMMFI_SITE_A || s.kind == MPGEMMFI_SITE_B) {
        const bool is_a = s.kind == MPGEMMFI_SITE_A;
        const size_t pos = (size_t)(is_a ? s.row : s.col) * p.K + s.k;
        const uint32_t before = load_operand(p.dtype, is_a ? p.A : p.Bt, pos);
        const uint32_t after = flip_operand(p.dtype, before, s.xor_mask);
        r.primary_index = (uint32_t)pos; r.before_bits = before; r.after_bits = after; r.final_bits = after;
        r.n_affected = is_a ? (uint32_t)p.N : (uint32_t)p.M;
        uint32_t *cnt = p.counters + (is_a ? 0 : 1);
        uint32_t *list = is_a ? p.list_a : p.list_b;
        list[atomicAdd(cnt, 1u)] = (uint32_t)t;
    } else {
        r.primary_index = s.row * (uint32_t)p.N + s.col;
        r.n_affected = 1;
        p.list_e[atomicAdd(p.counters + 2, 1u)] = (uint32_t)t;
    }
    p.records[t] = r;
}

// ---------------------------------------------------------------- single-element trials (one warp each)

__global__ void __launch_bounds__(256) element_kernel(CampaignParams p)
{
    const int lane = threadIdx.x & 31;
    const uint32_t warp_global = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t n_warps = (gridDim.x * blockDim.x) >> 5;
    const uint32_t count = p.counters[2];
    // granularity of a TERM write-back: the GEMM kernel's k-step, or one HMMA's worth of terms
    const uint32_t ks = (p.detect_mode & MPGEMMFI_TERM_HMMA_STEP) ? (p.dtype == MPGEMMFI_TF32 ? 8u : 16u)
                                                                  : (uint32_t)kstep_of(p.dtype);
    for (uint32_t w = warp_global; w < count; w += n_warps) {
        const uint32_t t = p.list_e[w];
        const mpgemmfi_site s = load_site(p.sites, t);
        const uint32_t lin = s.row * (uint32_t)p.N + s.col;
        uint32_t before, after, value_bits, clean_bits;
        if (s.kind == MPGEMMFI_SITE_OUT) {
            clean_bits = f32_bits(p.C[lin]);
            before = clean_bits;
            after = before ^ s.xor_mask;
            value_bits = after;
        } else {
            // where the site takes effect, in accumulated k elements
            uint32_t kb;
            float re2 = 0.0f, a_site = 0.0f, b_site = 0.0f;
            if (s.kind == MPGEMMFI_SITE_ACC) kb = s.k;
            else {
                kb = min((uint32_t)p.K, (s.k / ks + 1u) * ks);
                a_site = widen_operand(p.dtype, load_operand(p.dtype, p.A, (size_t)s.row * p.K + s.k));
                b_site = widen_operand(p.dtype, load_operand(p.dtype, p.Bt, (size_t)s.col * p.K + s.k));
                re2 = __fmul_rn(a_site, b_site);
            }
            float acc_c = 0.0f, acc_f = 0.0f;
            before = 0; after = 0;
            // Chunks of 128 terms: lane l holds terms k0 + 4 l .. k0 + 4 l + 3 (one 16- or 8-byte load per
            // operand), fetched two chunks ahead of their use: the rows come from L2 or HBM, a microsecond
            // away, and with a single 32-term chunk in flight that latency was the whole run time of a trial.
            const bool wide = p.dtype == MPGEMMFI_TF32;
            const unsigned char *a_row = reinterpret_cast<const unsigned char *>(p.A) + (size_t)s.row * p.K * (wide ? 4 : 2);
            const unsigned char *b_row = reinterpret_cast<const unsigned char *>(p.Bt) + (size_t)s.col * p.K * (wide ? 4 : 2);
            struct Raw { uint32_t a[4], b[4]; };
            auto fetch = [&](uint32_t k0, Raw &r) {
                const uint32_t k = k0 + 4u * (uint32_t)lane;
                r.a[0] = r.a[1] = r.a[2] = r.a[3] = 0u;
                r.b[0] = r.b[1] = r.b[2] = r.b[3] = 0u;
                if (k >= (uint32_t)p.K) return;            // K is a multiple of 4 (16-byte rows): groups of 4 are whole
                if (wide) {
                    const uint4 x = __ldg(reinterpret_cast<const uint4 *>(a_row) + (k >> 2));
                    const uint4 y = __ldg(reinterpret_cast<const uint4 *>(b_row) + (k >> 2));
                    r.a[0] = x.x; r.a[1] = x.y; r.a[2] = x.z; r.a[3] = x.w;
                    r.b[0] = y.x; r.b[1] = y.y; r.b[2] = y.z; r.b[3] = y.w;
                } else {
                    const uint2 x = __ldg(reinterpret_cast<const uint2 *>(a_row) + (k >> 2));
                    const uint2 y = __ldg(reinterpret_cast<const uint2 *>(b_row) + (k >> 2));
                    r.a[0] = x.x & 0xFFFFu; r.a[1] = x.x >> 16; r.a[2] = x.y & 0xFFFFu; r.a[3] = x.y >> 16;
                    r.b[0] = y.x & 0xFFFFu; r.b[1] = y.x >> 16; r.b[2] = y.y & 0xFFFFu; r.b[3] = y.y >> 16;
                }
            };
            auto site_hook = [&]() {
                if (s.kind == MPGEMMFI_SITE_ACC) {
                    before = f32_bits(acc_f);
                    after = before ^ s.xor_mask;
                    acc_f = bits_f32(after);
                } else if (p.detect_mode & MPGEMMFI_TERM_IN_FORMAT) {
                    // the product as a word of the operand format: rounded to it, flipped there, widened back; Eq. 1-2
                    // with this re_2 and its flipped version
                    before = round_to_operand(p.dtype, re2);
                    after = flip_operand(p.dtype, before, s.xor_mask);
                    const float re2_n = widen_operand(p.dtype, before);
                    bool det;
                    const uint32_t fin = product_check(p.detect_mode, f32_bits(widen_operand(p.dtype, after)), f32_bits(a_site),
                                                       f32_bits(b_site), det);
                    acc_f = __fadd_rn(__fsub_rn(acc_f, re2_n), bits_f32(fin));
                } else {
                    before = f32_bits(re2);
                    after = before ^ s.xor_mask;
                    bool det;
                    const uint32_t fin = product_check(p.detect_mode, after, f32_bits(a_site), f32_bits(b_site), det);
                    acc_f = __fadd_rn(__fsub_rn(acc_f, re2), bits_f32(fin));
                }
            };
            Raw r0, r1, r2;
            fetch(0, r0);
            fetch(128, r1);
            for (uint32_t k0 = 0; k0 < (uint32_t)p.K; k0 += 128) {
                fetch(k0 + 256, r2);
                float pr[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) pr[q] = __fmul_rn(widen_operand(p.dtype, r0.a[q]), widen_operand(p.dtype, r0.b[q]));
                const uint32_t n_here = min(128u, (uint32_t)p.K - k0);
                if (n_here == 128 && (kb <= k0 || kb > k0 + 128)) {
                    // whole chunk, the site does not fall inside it: straight-line additions in k order
#pragma unroll
                    for (uint32_t j = 0; j < 32; ++j) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float pj = __shfl_sync(0xFFFFFFFFu, pr[q], j);
                            acc_c = __fadd_rn(acc_c, pj);
                            acc_f = __fadd_rn(acc_f, pj);
                        }
                    }
                } else {
                    for (uint32_t t4 = 0; t4 < n_here; t4 += 4) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float pj = __shfl_sync(0xFFFFFFFFu, pr[q], t4 >> 2);
                            acc_c = __fadd_rn(acc_c, pj);
                            acc_f = __fadd_rn(acc_f, pj);
                            if (k0 + t4 + (uint32_t)q + 1 == kb) site_hook();
                        }
                    }
                }
                r0 = r1; r1 = r2;
            }
            clean_bits = f32_bits(acc_c);
            value_bits = f32_bits(acc_f);
        }
        if (lane == 0) {
            Stats st;
            stats_init(st);
            const uint32_t fin = stats_account(st, p.detect_mode, value_bits, clean_bits, lin);
            mpgemmfi_trial_record *r = &p.records[t];
            r->before_bits = before; r->after_bits = after; r->final_bits = fin;
            r->n_detected = st.n_det; r->idx_hash = st.hash; r->first_detected = st.first;
            r->max_abs_dev = bits_f32(st.maxdev_bits);
            r->status = status_bits(st, p.detect_mode);
        }
    }
}

// ---------------------------------------------------------------- operand trials (one CTA each)

// A-site trials (row i fixed, walk the N columns) and, when with_b is set, B-site trials (column j
// fixed, walk the M rows) in one launch: one CTA per trial, the A list first.
// Eq. 1-2 on a finished sum c for an operand trial: remove the clean product x * y, add the faulty one xf * y,
// every product and every sum rounded to FP32. The product of two FP16 values is exact in FP32 (22 significant
// bits, magnitudes between 2^-48 and 2^32, so neither underflow nor overflow), and then a fused multiply-add
// rounds once exactly where the separate sum would: the same bits (infinities, NaNs and signed zeros included)
// for half the instructions. BF16 and TF32 products can leave FP32's range and keep the separate operations.
__device__ __forceinline__ float operand_write_back(bool fp16, float c, float y, float x, float xf)
{
    if (fp16) return __fmaf_rn(xf, y, __fmaf_rn(-x, y, c));
    return __fadd_rn(__fsub_rn(c, __fmul_rn(x, y)), __fmul_rn(xf, y));
}

__global__ void __launch_bounds__(VEC_THREADS) vector_kernel(CampaignParams p, int with_b)
{
    __shared__ Stats warp_stats[VEC_THREADS / 32];
    const uint32_t count_a = p.counters[0];
    const uint32_t count = count_a + (with_b ? p.counters[1] : 0u);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t w = blockIdx.x; w < count; w += gridDim.x) {
        const bool is_a = w < count_a;
        const uint32_t t = is_a ? p.list_a[w] : p.list_b[w - count_a];
        const mpgemmfi_site s = load_site(p.sites, t);
        const size_t pos = (size_t)(is_a ? s.row : s.col) * p.K + s.k;
        const uint32_t w_clean = load_operand(p.dtype, is_a ? p.A : p.Bt, pos);
        const float x = widen_operand(p.dtype, w_clean);
        const float xf = widen_operand(p.dtype, flip_operand(p.dtype, w_clean, s.xor_mask));
        const uint32_t n_other = is_a ? (uint32_t)p.N : (uint32_t)p.M;
        const void *other = is_a ? p.Bt : p.A;
        Stats st;
        stats_init(st);
        // four elements per thread and round: their (strided, L2-latency-bound) loads are all in flight
        // before the first is used
        constexpr int UNROLL = 4;
        for (uint32_t o0 = threadIdx.x; o0 < n_other; o0 += UNROLL * VEC_THREADS) {
            uint32_t yw[UNROLL];
            float c[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t o = o0 + (uint32_t)(u * VEC_THREADS);
                if (o < n_other) {
                    yw[u] = load_operand(p.dtype, other, (size_t)o * p.K + s.k);
                    c[u] = p.C[is_a ? s.row * (uint32_t)p.N + o : o * (uint32_t)p.N + s.col];
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const uint32_t o = o0 + (uint32_t)(u * VEC_THREADS);
                if (o < n_other) {
                    const float y = widen_operand(p.dtype, yw[u]);
                    const uint32_t lin = is_a ? s.row * (uint32_t)p.N + o : o * (uint32_t)p.N + s.col;
                    const float cf = operand_write_back(p.dtype == MPGEMMFI_FP16, c[u], y, x, xf);     // Eq. 1, Eq. 2
                    stats_account(st, p.detect_mode, f32_bits(cf), f32_bits(c[u]), lin);
                }
            }
        }
        stats_warp_reduce(st);
        if (lane == 0) warp_stats[warp] = st;
        __syncthreads();
        if (threadIdx.x == 0) {
            Stats tot = warp_stats[0];
            for (int i = 1; i < VEC_THREADS / 32; ++i) {
                tot.n_det += warp_stats[i].n_det;
                tot.first = min(tot.first, warp_stats[i].first);
                tot.maxdev_bits = max(tot.maxdev_bits, warp_stats[i].maxdev_bits);
                tot.changed |= warp_stats[i].changed;
                tot.hash += warp_stats[i].hash;
            }
            mpgemmfi_trial_record *r = &p.records[t];
            r->n_detected = tot.n_det; r->idx_hash = tot.hash; r->first_detected = tot.first;
            r->max_abs_dev = bits_f32(tot.maxdev_bits);
            r->status = status_bits(tot, p.detect_mode);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------- B-site trials, batched by row panel

// When a row panel of A (R rows x K) and of C (R rows x N) fits in shared memory, B-site trials
// are evaluated panel by panel: a CTA loads a panel once and applies a whole group of trials to
// it, so A and C are streamed once per GROUP of trials instead of once per trial (each trial
// alone would pull one 32-byte sector per row out of both matrices).
// Work item = (group of up to PANEL_GROUP trials) x (contiguous chunk of panels); a thread keeps its
// trial's partial statistics in registers and merges them into the record with atomics at the end.
constexpr int PANEL_GROUP = 1024;
constexpr int PANEL_THREADS = 1024;

struct PanelShape {
    int rows;        // R, rows of one staged panel (two panels are resident: one evaluated, one arriving), multiple of 8
    int a_words;     // 32-bit words per staged A row (the row as it is in global memory: K * element size / 4)
    int c_words;     // 32-bit words per staged C row (N)
    size_t smem;
};

__host__ __device__ inline PanelShape panel_shape(int dtype, int N, int K, size_t smem_limit)
{
    PanelShape s;
    s.a_words = K * esize_of(dtype) / 4;       // K * element size is a multiple of 16 bytes
    s.c_words = N;
    const size_t fixed = (size_t)PANEL_GROUP * (6 * 4) + 256;    // trial parameters and sort keys
    const size_t row_bytes = 4 * (size_t)(s.a_words + s.c_words);
    long long r = smem_limit > fixed ? (long long)((smem_limit - fixed) / (2 * row_bytes)) : 0;
    r = r / 8 * 8;
    if (r > 128) r = 128;
    s.rows = (int)r;
    s.smem = fixed + 2 * row_bytes * (size_t)(r > 0 ? r : 0);
    return s;
}

// One thread per trial of the group (PANEL_GROUP == PANEL_THREADS): it walks the rows of the staged panel
// with its own column j of C and its own element k of every A row, and keeps its trial's statistics in
// registers over the whole chunk of panels -- no warp-wide reduction, one merge into the record per item.
// The trials of a group are ordered by k first, so that the threads of a warp read the same or
// neighbouring words of an A row (broadcast, or distinct banks) instead of 32 random ones.
// asynchronous global -> shared copies (LSU path, no registers in between), grouped per panel
__device__ __forceinline__ void cp_async_16(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}

__device__ __forceinline__ void cp_async_4(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst_smem), "l"(src) : "memory");
}

__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all_but_one() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }

// 32-bit word of shared memory at a 32-bit shared-space address (address arithmetic stays 32-bit)
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// 16-bit word of shared memory, zero-extended
__device__ __forceinline__ uint32_t lds_u16(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

template <int kDtype>
__device__ __forceinline__ void panel_rows(const uint32_t *As, const uint32_t *Cs, const PanelShape &ps, uint32_t rows,
                                           uint32_t lin_base, uint32_t n_cols, uint32_t j, uint32_t k, float b, float bf,
                                           bool do_bound, bool do_corr, uint32_t &n_det, uint32_t &first,
                                           unsigned long long &hash, float &maxdev, uint32_t &changed)
{
    constexpr bool two_byte = kDtype != MPGEMMFI_TF32;
    // the trial's element of the first row: a 16-bit or a 32-bit word
    uint32_t a_addr = (uint32_t)__cvta_generic_to_shared(As) + (two_byte ? 2u : 4u) * k;
    uint32_t c_addr = (uint32_t)__cvta_generic_to_shared(Cs + j);
    auto lds_a = [](uint32_t addr) { return two_byte ? lds_u16(addr) : lds_u32(addr); };
    const uint32_t a_step = 4u * (uint32_t)ps.a_words, c_step = 4u * (uint32_t)ps.c_words;

    // one row, every case handled (flagged values, infinities, NaNs)
    auto exact_row = [&](uint32_t r, uint32_t aw, uint32_t c_bits) {
        const float a = widen_operand(kDtype, aw);
        const float c = bits_f32(c_bits);
        const float cf = operand_write_back(kDtype == MPGEMMFI_FP16, c, a, b, bf);      // Eq. 1, Eq. 2 on the finished sum
        uint32_t fin = f32_bits(cf);
        if (do_bound && !(fabsf(cf) < 131072.0f)) {               // exponent field >= 0x90
            const uint32_t lin = lin_base + r * n_cols;
            ++n_det;
            hash += ((unsigned long long)lin + 1ull) * HASH_MUL;
            first = min(first, lin);
            if (do_corr) fin = boundcheck_clear(fin);
        }
        changed |= fin ^ c_bits;
        const float d = fabsf(__fsub_rn(bits_f32(fin), c));
        maxdev = d != d ? __uint_as_float(0x7F800000u) : fmaxf(maxdev, d);      // a NaN deviation counts as +inf
    };

    constexpr int STEP = 8;
    uint32_t r = 0;
    for (; r + STEP <= rows; r += STEP, a_addr += STEP * a_step, c_addr += STEP * c_step) {
        // STEP rows at once on the assumption that nothing is flagged and nothing is infinite or NaN (one
        // compare per row, folded into one branch per step); otherwise the rows are done again, exactly.
        uint32_t aw[STEP], cb[STEP];
#pragma unroll
        for (int u = 0; u < STEP; ++u) { aw[u] = lds_a(a_addr + u * a_step); cb[u] = lds_u32(c_addr + u * c_step); }
        bool plain = true;
        uint32_t ch = 0;
        float md = 0.0f;
#pragma unroll
        for (int u = 0; u < STEP; ++u) {
            const float a = widen_operand(kDtype, aw[u]);
            const float c = bits_f32(cb[u]);
            const float cf = operand_write_back(kDtype == MPGEMMFI_FP16, c, a, b, bf);       // Eq. 1, Eq. 2
            plain = plain && (fabsf(cf) < 131072.0f);
            ch |= f32_bits(cf) ^ cb[u];
            md = fmaxf(md, fabsf(__fsub_rn(cf, c)));        // cf finite and below the bound: never NaN (c is finite too)
        }
        if (plain) {
            changed |= ch;
            maxdev = fmaxf(maxdev, md);
        } else {
#pragma unroll
            for (int u = 0; u < STEP; ++u) exact_row(r + u, aw[u], cb[u]);
        }
    }
    for (; r < rows; ++r, a_addr += a_step, c_addr += c_step) exact_row(r, lds_a(a_addr), lds_u32(c_addr));
}

__global__ void __launch_bounds__(PANEL_THREADS) panel_kernel(CampaignParams p, PanelShape ps)
{
    static_assert(PANEL_GROUP == PANEL_THREADS, "one thread per trial of a group");
    extern __shared__ __align__(16) unsigned char panel_smem[];
    // two panels: A rows of both (16-byte aligned), then C rows of both
    uint32_t *As2 = reinterpret_cast<uint32_t *>(panel_smem);
    uint32_t *Cs2 = As2 + 2 * (size_t)ps.rows * ps.a_words;
    uint32_t *t_id = Cs2 + 2 * (size_t)ps.rows * ps.c_words;
    uint32_t *t_j = t_id + PANEL_GROUP;
    uint32_t *t_k = t_j + PANEL_GROUP;
    float *t_b = reinterpret_cast<float *>(t_k + PANEL_GROUP);
    float *t_bf = t_b + PANEL_GROUP;
    uint32_t *t_key = reinterpret_cast<uint32_t *>(t_bf + PANEL_GROUP);

    const uint32_t count = p.counters[1];
    if (count == 0) return;
    const uint32_t tid = threadIdx.x;
    const int es = esize_of(p.dtype);
    const uint32_t n_groups = (count + PANEL_GROUP - 1) / PANEL_GROUP;
    const uint32_t n_panels = ((uint32_t)p.M + ps.rows - 1) / ps.rows;
    // enough items to occupy the grid about twice over, but never fewer than 4 panels per item
    uint32_t n_chunks = (2 * gridDim.x + n_groups - 1) / n_groups;
    n_chunks = max(1u, min(n_chunks, (n_panels + 3) / 4));
    const uint32_t panels_per_chunk = (n_panels + n_chunks - 1) / n_chunks;
    const bool do_bound = (p.detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK) == MPGEMMFI_DETECT_BOUNDCHECK;
    const bool do_corr = do_bound && (p.detect_mode & MPGEMMFI_CORRECT);

    for (uint32_t item = blockIdx.x; item < n_groups * n_chunks; item += gridDim.x) {
        const uint32_t g = item / n_chunks, ch = item % n_chunks;
        const uint32_t g_beg = g * PANEL_GROUP, g_n = min((uint32_t)PANEL_GROUP, count - g_beg);
        __syncthreads();                       // the tables of the previous item are no longer read
        // the group's trials, ordered by k (rank by counting: g_n <= 1024 keys in shared memory)
        {
            uint32_t t = 0, j = 0, k = 0xFFFFFFFFu;
            float b = 0.0f, bf = 0.0f;
            if (tid < g_n) {
                t = p.list_b[g_beg + tid];
                const mpgemmfi_site s = load_site(p.sites, t);
                const uint32_t w_clean = load_operand(p.dtype, p.Bt, (size_t)s.col * p.K + s.k);
                j = s.col; k = s.k;
                b = widen_operand(p.dtype, w_clean);
                bf = widen_operand(p.dtype, flip_operand(p.dtype, w_clean, s.xor_mask));
            }
            t_key[tid] = k;
            __syncthreads();
            if (tid < g_n) {
                uint32_t rank = 0;
                for (uint32_t i = 0; i < g_n; ++i) {
                    const uint32_t ki = t_key[i];
                    rank += (ki < k || (ki == k && i < tid)) ? 1u : 0u;
                }
                t_id[rank] = t; t_j[rank] = j; t_k[rank] = k; t_b[rank] = b; t_bf[rank] = bf;
            }
            __syncthreads();
        }
        const bool have = tid < g_n;
        const uint32_t my_t = have ? t_id[tid] : 0u, my_j = have ? t_j[tid] : 0u, my_k = have ? t_k[tid] : 0u;
        const float my_b = have ? t_b[tid] : 0.0f, my_bf = have ? t_bf[tid] : 0.0f;
        uint32_t n_det = 0, first = 0xFFFFFFFFu, changed = 0;
        float maxdev = 0.0f;                   // non-negative or +inf
        unsigned long long hash = 0ull;

        const uint32_t p_beg = ch * panels_per_chunk, p_end = min(n_panels, p_beg + panels_per_chunk);
        // Panel pn of A and C into buffer `buf`, asynchronously (cp.async, one group per panel). A panel's rows
        // are contiguous in global memory and are kept that way in shared memory: a flat copy in 16-byte pieces
        // (4-byte pieces for C when its panel does not start or end on a 16-byte boundary).
        auto stage = [&](uint32_t pn, uint32_t buf) {
            const uint32_t row0 = pn * (uint32_t)ps.rows;
            if (row0 >= (uint32_t)p.M) return;                 // no such panel: nothing to copy
            const uint32_t rows = min((uint32_t)ps.rows, (uint32_t)p.M - row0);
            const unsigned char *Ag = reinterpret_cast<const unsigned char *>(p.A) + (size_t)row0 * p.K * es;
            const uint32_t a_dst = (uint32_t)__cvta_generic_to_shared(As2 + (size_t)buf * ps.rows * ps.a_words);
            const uint32_t a_pieces = rows * (uint32_t)ps.a_words / 4;
            for (uint32_t i = tid; i < a_pieces; i += PANEL_THREADS) cp_async_16(a_dst + 16 * i, Ag + 16 * (size_t)i);
            const float *Cg = p.C + (size_t)row0 * p.N;
            const uint32_t c_dst = (uint32_t)__cvta_generic_to_shared(Cs2 + (size_t)buf * ps.rows * ps.c_words);
            const uint32_t c_words = rows * (uint32_t)p.N;
            if (((reinterpret_cast<uintptr_t>(Cg) | c_words * 4u) & 15u) == 0) {
                for (uint32_t i = tid; i < c_words / 4; i += PANEL_THREADS) cp_async_16(c_dst + 16 * i, Cg + 4 * (size_t)i);
            } else {
                for (uint32_t i = tid; i < c_words; i += PANEL_THREADS) cp_async_4(c_dst + 4 * i, Cg + i);
            }
            cp_async_commit();
        };
        __syncthreads();           // nobody still reads the panels of the previous item
        // (the chunk count is rounded up: the last items of a launch may have no panel at all)
        if (p_beg < p_end) stage(p_beg, 0);
        for (uint32_t pn = p_beg; pn < p_end; ++pn) {
            const uint32_t buf = (pn - p_beg) & 1u;
            const uint32_t row0 = pn * (uint32_t)ps.rows;
            const uint32_t rows = min((uint32_t)ps.rows, (uint32_t)p.M - row0);
            // the next panel starts to arrive in the other buffer (last read two panels ago) ...
            if (pn + 1 < p_end) { stage(pn + 1, buf ^ 1u); cp_async_wait_all_but_one(); }
            else cp_async_wait_all();
            __syncthreads();       // ... and this one is complete for every thread
            if (have) {
                const uint32_t *As = As2 + (size_t)buf * ps.rows * ps.a_words;
                const uint32_t *Cs = Cs2 + (size_t)buf * ps.rows * ps.c_words;
                const uint32_t lin_base = row0 * (uint32_t)p.N + my_j;
                if (p.dtype == MPGEMMFI_FP16)
                    panel_rows<MPGEMMFI_FP16>(As, Cs, ps, rows, lin_base, (uint32_t)p.N, my_j, my_k, my_b, my_bf, do_bound, do_corr, n_det, first, hash, maxdev, changed);
                else if (p.dtype == MPGEMMFI_BF16)
                    panel_rows<MPGEMMFI_BF16>(As, Cs, ps, rows, lin_base, (uint32_t)p.N, my_j, my_k, my_b, my_bf, do_bound, do_corr, n_det, first, hash, maxdev, changed);
                else
                    panel_rows<MPGEMMFI_TF32>(As, Cs, ps, rows, lin_base, (uint32_t)p.N, my_j, my_k, my_b, my_bf, do_bound, do_corr, n_det, first, hash, maxdev, changed);
            }
            __syncthreads();       // this buffer may be overwritten by the panel after the next
        }
        // merge this item's statistics into the trial's record
        if (have) {
            mpgemmfi_trial_record *r = &p.records[my_t];
            const uint32_t maxdev_bits = f32_bits(maxdev);     // non-negative floats order like their bit patterns
            if (n_det) {
                atomicAdd(&r->n_detected, n_det);
                atomicAdd(reinterpret_cast<unsigned long long *>(&r->idx_hash), hash);
                atomicMin(&r->first_detected, first);
            }
            if (maxdev_bits) atomicMax(reinterpret_cast<uint32_t *>(&r->max_abs_dev), maxdev_bits);
            const uint32_t st = (changed ? 1u : 0u) | (n_det ? 2u : 0u) | ((n_det && do_corr) ? 4u : 0u);
            if (st) atomicOr(&r->status, st);
        }
    }
}

// ---------------------------------------------------------------- deviation summary

__global__ void __launch_bounds__(256) summary_kernel(const mpgemmfi_trial_record *records, int n, mpgemmfi_summary *out)
{
    __shared__ uint32_t hist[256];
    __shared__ uint32_t cnt[16];      // 0 invalid, 1 zero-diff, 2 detected, 3 corrected, 4 non-finite, 5.. unused
    __shared__ uint32_t kind_trials[5], kind_zero[5];
    for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
    if (threadIdx.x < 16) cnt[threadIdx.x] = 0;
    if (threadIdx.x < 5) { kind_trials[threadIdx.x] = 0; kind_zero[threadIdx.x] = 0; }
    __syncthreads();
    for (int t = blockIdx.x * blockDim.x + threadIdx.x; t < n; t += gridDim.x * blockDim.x) {
        const mpgemmfi_trial_record r = records[t];
        if (r.status & (1u << 8)) { atomicAdd(&cnt[0], 1u); continue; }
        const bool zero = (r.status & 1u) == 0;
        if (zero) atomicAdd(&cnt[1], 1u);
        if (r.status & 2u) atomicAdd(&cnt[2], 1u);
        if (r.status & 4u) atomicAdd(&cnt[3], 1u);
        if (r.kind < 5) { atomicAdd(&kind_trials[r.kind], 1u); if (zero) atomicAdd(&kind_zero[r.kind], 1u); }
        uint32_t d = f32_bits(r.max_abs_dev) & 0x7FFFFFFFu;
        if (d > 0x7F800000u) d = 0x7F800000u;                      // NaN counts as infinite
        if (d == 0x7F800000u) atomicAdd(&cnt[4], 1u);
        if (d != 0) atomicAdd(&hist[d >> 23], 1u);
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 256; i += blockDim.x)
        if (hist[i]) atomicAdd(&out->dev_exponent_hist[i], hist[i]);
    if (threadIdx.x == 0) {
        if (blockIdx.x == 0) out->n_trials = (uint32_t)n;
        if (cnt[0]) atomicAdd(&out->n_invalid, cnt[0]);
        if (cnt[1]) atomicAdd(&out->n_zero_diff, cnt[1]);
        if (cnt[2]) atomicAdd(&out->n_detected, cnt[2]);
        if (cnt[3]) atomicAdd(&out->n_corrected, cnt[3]);
        if (cnt[4]) atomicAdd(&out->n_nonfinite, cnt[4]);
        for (int k = 0; k < 5; ++k) {
            if (kind_trials[k]) atomicAdd(&out->kind_trials[k], kind_trials[k]);
            if (kind_zero[k]) atomicAdd(&out->kind_zero_diff[k], kind_zero[k]);
        }
    }
}

}  // namespace

cudaError_t launch_campaign_summary(const mpgemmfi_trial_record *records, int n_trials, mpgemmfi_summary *out,
                                    int num_sms, cudaStream_t stream)
{
    cudaError_t e = cudaMemsetAsync(out, 0, sizeof(mpgemmfi_summary), stream);
    if (e != cudaSuccess) return e;
    const int grid = max(1, min((n_trials + 255) / 256, 4 * num_sms));
    summary_kernel<<<grid, 256, 0, stream>>>(records, n_trials, out);
    return cudaGetLastError();
}

size_t campaign_schedule_bytes(int n_trials)
{
    const size_t lists = 3 * sizeof(uint32_t) * (size_t)(n_trials > 0 ? n_trials : 0);
    return (256 + lists + 255) / 256 * 256;
}

void campaign_bind_schedule(CampaignParams &p, void *scratch)
{
    uint32_t *w = static_cast<uint32_t *>(scratch);
    p.counters = w;
    p.list_a = w + 64;
    p.list_b = p.list_a + p.n_trials;
    p.list_e = p.list_b + p.n_trials;
}

// Built-in schedule scratch for callers that cannot allocate device memory. It lives in every
// context that loads the library, for as long as the library stays loaded.
static __device__ __align__(256) unsigned char g_static_schedule[256 + 3 * sizeof(uint32_t) * CAMPAIGN_STATIC_MAX_TRIALS];

cudaError_t campaign_static_schedule(void **ptr, size_t *bytes)
{
    // In host code `g_static_schedule` is only a handle for the runtime; the address a kernel can
    // use has to be asked for, once per device, while that device is current.
    static void *addr[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    void *a = (dev >= 0 && dev < 64) ? addr[dev] : nullptr;
    if (!a) {
        e = cudaGetSymbolAddress(&a, g_static_schedule);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) addr[dev] = a;
    }
    *ptr = a;
    *bytes = sizeof(g_static_schedule);
    return cudaSuccess;
}

cudaError_t launch_campaign_trials(const CampaignParams &p, int num_sms, cudaStream_t stream)
{
    if (p.n_trials <= 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(p.counters, 0, 256, stream);
    if (e != cudaSuccess) return e;
    schedule_kernel<<<(p.n_trials + 255) / 256, 256, 0, stream>>>(p);
    const int max_ctas = num_sms * 8;
    const int grid_e = min((p.n_trials + 7) / 8, max_ctas);
    element_kernel<<<grid_e, 256, 0, stream>>>(p);
    const int grid_v = min(p.n_trials, max_ctas);
    // B-site trials: by row panel when a useful panel fits in shared memory and the columns are long;
    // otherwise one CTA per trial, in the same launch as the A-site trials
    const PanelShape ps = panel_shape(p.dtype, p.N, p.K, 227 * 1024);
    const bool by_panel = ps.rows >= 32 && p.M >= 16 * ps.rows;
    vector_kernel<<<grid_v, VEC_THREADS, 0, stream>>>(p, by_panel ? 0 : 1);
    if (by_panel) {
        static bool configured[64] = {};
        int dev = 0;
        e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64 || !configured[dev]) {
            e = cudaFuncSetAttribute(panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) configured[dev] = true;
        }
        panel_kernel<<<num_sms, PANEL_THREADS, ps.smem, stream>>>(p, ps);
    }
    return cudaGetLastError();
}

}  // namespace mpg
