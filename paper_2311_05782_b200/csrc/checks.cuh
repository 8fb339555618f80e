// Device/host helpers: operand formats, fault-site validity and the exponent-only
// checks (paper Section II-A, Section VI-A, Table III).
#pragma once

#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "../../include/mpgemmfi.h"

namespace mpg {

#define MPG_HD __host__ __device__ __forceinline__

__device__ __forceinline__ uint32_t f32_bits(float f) { return __float_as_uint(f); }
__device__ __forceinline__ float bits_f32(uint32_t u) { return __uint_as_float(u); }

MPG_HD int kstep_of(int dtype) { return dtype == MPGEMMFI_TF32 ? 32 : 64; }
// log2 of the k-step (the k-step is a power of two: shifts instead of integer divisions on the device)
MPG_HD uint32_t kshift_of(int dtype) { return dtype == MPGEMMFI_TF32 ? 5u : 6u; }
MPG_HD int esize_of(int dtype) { return dtype == MPGEMMFI_TF32 ? 4 : 2; }

// XOR a mask into an operand storage word. 16-bit formats: mask bits 0..15.
// TF32: mask bit b (0..18) is bit b+13 of the 32-bit word.
MPG_HD uint32_t flip_operand(int dtype, uint32_t s, uint32_t mask)
{
    if (dtype == MPGEMMFI_TF32) return (s & 0xFFFFE000u) ^ ((mask & 0x7FFFFu) << 13);
    return (s & 0xFFFFu) ^ (mask & 0xFFFFu);
}

// storage word -> FP32 value (exact in all three formats)
__device__ __forceinline__ float widen_operand(int dtype, uint32_t s)
{
    if (dtype == MPGEMMFI_BF16) return __uint_as_float(s << 16);
    if (dtype == MPGEMMFI_TF32) return __uint_as_float(s & 0xFFFFE000u);
    return __half2float(__ushort_as_half(static_cast<unsigned short>(s)));
}

// FP32 value -> storage word of the operand format, round to nearest even (FP16 / BF16: the conversion
// instructions; TF32: on the 13 dropped bits of the FP32 word, Inf kept, NaN kept a NaN)
__device__ __forceinline__ uint32_t round_to_operand(int dtype, float v)
{
    if (dtype == MPGEMMFI_FP16) return __half_as_ushort(__float2half_rn(v));
    if (dtype == MPGEMMFI_BF16) return __bfloat16_as_ushort(__float2bfloat16_rn(v));
    const uint32_t u = __float_as_uint(v);
    if (((u >> 23) & 0xFFu) == 0xFFu) return (u & 0xFFFFE000u) | ((u & 0x7FFFFFu) ? 0x00400000u : 0u);
    const uint32_t keep = u >> 13, rest = u & 0x1FFFu;
    return (keep + ((rest > 0x1000u || (rest == 0x1000u && (keep & 1u))) ? 1u : 0u)) << 13;
}

__device__ __forceinline__ uint32_t load_operand(int dtype, const void *base, size_t idx)
{
    if (dtype == MPGEMMFI_TF32) return __ldg(reinterpret_cast<const uint32_t *>(base) + idx) & 0xFFFFE000u;
    return __ldg(reinterpret_cast<const unsigned short *>(base) + idx);
}

// Same rules on host (mpgemmfi_validate_sites) and device (bad entries are skipped).
MPG_HD bool site_valid(const mpgemmfi_site &s, int dtype, int M, int N, int K)
{
    const uint32_t ks = static_cast<uint32_t>(kstep_of(dtype));
    switch (s.kind) {
    case MPGEMMFI_SITE_A: return s.row < (uint32_t)M && s.k < (uint32_t)K;
    case MPGEMMFI_SITE_B: return s.col < (uint32_t)N && s.k < (uint32_t)K;
    case MPGEMMFI_SITE_ACC:
        return s.row < (uint32_t)M && s.col < (uint32_t)N && s.k >= 1 && s.k <= (uint32_t)K &&
               ((s.k & (ks - 1u)) == 0 || s.k == (uint32_t)K);
    case MPGEMMFI_SITE_OUT: return s.row < (uint32_t)M && s.col < (uint32_t)N;
    case MPGEMMFI_SITE_TERM: return s.row < (uint32_t)M && s.col < (uint32_t)N && s.k < (uint32_t)K;
    default: return false;
    }
}

// Number of whole k-steps accumulated when a site takes effect (ACC, TERM).
MPG_HD uint32_t site_boundary(const mpgemmfi_site &s, int dtype, int K)
{
    const uint32_t ks = static_cast<uint32_t>(kstep_of(dtype));
    const uint32_t sh = kshift_of(dtype);
    const uint32_t nkt = ((uint32_t)K + ks - 1) >> sh;
    if (s.kind == MPGEMMFI_SITE_ACC) return s.k == (uint32_t)K ? nkt : s.k >> sh;
    return (s.k >> sh) + 1;   // TERM: the boundary that ends the k-step containing k
}

// ---- BoundCheck: exponent bit 7 set and any of exponent bits 6..4 set ("1eeexxxx"), i.e. an
// exponent field of 0x90 or more: the magnitude bits are at least those of 131072.0f
MPG_HD bool boundcheck_detect(uint32_t bits)
{
    return (bits & 0x7FFFFFFFu) >= 0x48000000u;
}
MPG_HD uint32_t boundcheck_clear(uint32_t bits) { return bits & ~0x38000000u; }

// ---- RangeCheck: biased exponent of a product is at most E1 + E2 - 126 (e_m <= e1 + e2 + 1)
MPG_HD int rangecheck_bound(uint32_t a_bits, uint32_t b_bits)
{
    int b = (int)((a_bits >> 23) & 0xFFu) + (int)((b_bits >> 23) & 0xFFu) - 126;
    return b < 0 ? 0 : (b > 255 ? 255 : b);
}
MPG_HD uint32_t rangecheck_max(uint32_t p, int bound)
{
    return (p & 0x807FFFFFu) | ((uint32_t)bound << 23);
}
MPG_HD uint32_t rangecheck_flip(uint32_t p, int bound)
{
    uint32_t E = (p >> 23) & 0xFFu;
#pragma unroll
    for (int b = 0; b < 8; ++b)
        if ((int)E > bound) E &= ~(1u << b);
    return (p & 0x807FFFFFu) | (E << 23);
}

// Check applied to a faulty product p_err = a*b ^ mask. Returns the (possibly corrected) bits.
MPG_HD uint32_t product_check(int detect_mode, uint32_t p_err, uint32_t a_bits, uint32_t b_bits, bool &det)
{
    const int tech = detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK;
    const bool corr = (detect_mode & MPGEMMFI_CORRECT) != 0;
    det = false;
    if (tech == MPGEMMFI_DETECT_BOUNDCHECK) {
        det = boundcheck_detect(p_err);
        return (det && corr) ? boundcheck_clear(p_err) : p_err;
    }
    if (tech == MPGEMMFI_DETECT_RANGE_MAX || tech == MPGEMMFI_DETECT_RANGE_FLIP) {
        const int bound = rangecheck_bound(a_bits, b_bits);
        det = (int)((p_err >> 23) & 0xFFu) > bound;
        if (det && corr) return tech == MPGEMMFI_DETECT_RANGE_MAX ? rangecheck_max(p_err, bound) : rangecheck_flip(p_err, bound);
    }
    return p_err;
}

// Check applied to an output element (BoundCheck only).
MPG_HD uint32_t output_check(int detect_mode, uint32_t bits, bool &det)
{
    det = false;
    if ((detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK) != MPGEMMFI_DETECT_BOUNDCHECK) return bits;
    det = boundcheck_detect(bits);
    return (det && (detect_mode & MPGEMMFI_CORRECT)) ? boundcheck_clear(bits) : bits;
}

__device__ __forceinline__ mpgemmfi_site load_site(const mpgemmfi_site *sites, int idx)
{
    const uint4 *p = reinterpret_cast<const uint4 *>(sites + idx);
    const uint4 lo = __ldg(p);
    const uint4 hi = __ldg(p + 1);
    mpgemmfi_site s;
    s.kind = lo.x; s.row = lo.y; s.col = lo.z; s.k = lo.w;
    s.xor_mask = hi.x; s.trial = hi.y; s.pad[0] = hi.z; s.pad[1] = hi.w;
    return s;
}

}  // namespace mpg
