// C ABI of the library: argument checks, tensor-map encoding, kernel launches.
#include <atomic>
#include <cstdint>
#include <cstring>
#include <cuda.h>
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include "../../include/mpgemmfi.h"
#include "campaign.cuh"
#include "checks.cuh"
#include "gemm_sm100.cuh"
#include "operands.cuh"

static_assert(MPGEMMFI_STATIC_MAX_TRIALS == mpg::CAMPAIGN_STATIC_MAX_TRIALS, "header and kernel limits differ");

namespace {

std::atomic<int> g_last_cuda_error{0};

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return MPGEMMFI_ERR_CUDA;
}

// NVTX range over the queueing of one part of a call (a profiler's timeline then shows the clean GEMM and the trial
// kernels of a campaign apart); a no-op when no tool is attached
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
    Range(const Range &) = delete;
    Range &operator=(const Range &) = delete;
};

struct DeviceInfo {
    bool known = false;
    int major = 0;
    int num_sms = 0;
};

// properties of the current device, looked up once per device
int device_info(DeviceInfo &out)
{
    static DeviceInfo cache[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e);
    if (dev < 0 || dev >= 64) return MPGEMMFI_ERR_ARG;
    if (!cache[dev].known) {
        e = cudaDeviceGetAttribute(&cache[dev].major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        e = cudaDeviceGetAttribute(&cache[dev].num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return cuda_fail(e);
        cache[dev].known = true;
    }
    out = cache[dev];
    return MPGEMMFI_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// rows x K matrix, K contiguous; box = one 128-byte row segment x box_rows rows, 128-byte swizzle,
// out-of-range elements read as zero
int encode_operand_map(CUtensorMap *map, int dtype, const void *base, int rows, int K, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return cuda_fail(cudaErrorUnknown);
    const int es = mpg::esize_of(dtype);
    const CUtensorMapDataType dt = dtype == MPGEMMFI_FP16   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                   : dtype == MPGEMMFI_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                            : CU_TENSOR_MAP_DATA_TYPE_FLOAT32;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)K * (cuuint64_t)es};
    const cuuint32_t box[2] = {(cuuint32_t)(128 / es), (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, dt, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return MPGEMMFI_ERR_CUDA; }
    return MPGEMMFI_OK;
}

// C as an M x N FP32 tensor; box = 32 columns (one 128-byte swizzle row) x 16 rows: what one epilogue warp
// hands to the TMA engine per store
int encode_output_map(CUtensorMap *map, float *C, int M, int N)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return cuda_fail(cudaErrorUnknown);
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)N * 4u};
    const cuuint32_t box[2] = {32, 16};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, C, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return MPGEMMFI_ERR_CUDA; }
    return MPGEMMFI_OK;
}

// the same for a 16-bit output (FP16 or BF16 words): box = 32 columns (64 bytes) x 32 rows, 64-byte swizzle: one
// whole 32 x 32 piece of an epilogue warp per store
int encode_output_map16(CUtensorMap *map, void *D, int out_fmt, int M, int N)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return cuda_fail(cudaErrorUnknown);
    const cuuint64_t dims[2] = {(cuuint64_t)N, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)N * 2u};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = out_fmt == MPGEMMFI_OUT_FP16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = fn(map, dt, 2, D, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { g_last_cuda_error = (int)r; return MPGEMMFI_ERR_CUDA; }
    return MPGEMMFI_OK;
}

// process-wide knobs: each is read once when a launch is queued; atomics, so that a host thread changing one while
// another queues a launch gives that launch either the old or the new value, never a torn one
std::atomic<int> g_tile_policy{MPGEMMFI_TILES_AUTO};
std::atomic<int> g_split_policy{MPGEMMFI_SPLIT_AUTO};
std::atomic<int> g_wait_limit_ms{4000};
std::atomic<int> g_break_handover{0};

}  // namespace

void mpg::choose_split_schedule(mpg::GemmParams &p, int walkers, int policy)
{
    p.split_parts = 0; p.full_rounds = 0; p.left_tiles = 0;
    // (a cut tile's unfinished FP32 sums wait in C: not with a 16-bit C)
    if (policy == MPGEMMFI_SPLIT_OFF || !p.c_vec_ok || p.out_fmt != MPGEMMFI_OUT_FP32) return;
    const int rounds = p.num_tiles / walkers, left = p.num_tiles % walkers;
    if (rounds < 1 || left == 0 || left * 16 > mpg::SPLIT_SIGNAL_WORDS) return;
    int parts = walkers / left;
    if (parts > 4) parts = 4;
    if (parts > rounds + 1) parts = rounds + 1;
    while (parts >= 2 && p.num_kt / parts < 4) --parts;
    if (parts < 2) return;
    if (policy == MPGEMMFI_SPLIT_AUTO) {
        // a cut tile costs its walkers one more pass of accumulators through C (measured: about 5 us); it
        // pays when the k-tiles saved (0.35 us each) outweigh that and are a visible share of the launch
        const int saved = p.num_kt - (p.num_kt + parts - 1) / parts;
        if (saved < 24 || saved < 0.03 * (rounds + 1) * p.num_kt) return;
    }
    p.split_parts = parts; p.full_rounds = rounds; p.left_tiles = left;
}

namespace {

// widest tile that still gives every SM a tile; narrow outputs get narrow tiles
int choose_bn(int M, int N, int num_sms)
{
    const int tiles_m = (M + 127) / 128;
    const int cands[3] = {256, 128, 64};
    for (int i = 0; i < 3; ++i) {
        const int bn = cands[i];
        if (i < 2 && N <= bn / 2) continue;                 // tile twice as wide as the matrix
        if (tiles_m * ((N + bn - 1) / bn) >= num_sms || i == 2) return bn;
    }
    return 64;
}

// 256 x 256 tiles on CTA pairs pay off once there are enough of them to occupy most pairs
bool choose_pair(int dtype, int M, int N, int *max_pairs)
{
    const int policy = g_tile_policy.load();
    if (policy == MPGEMMFI_TILES_SINGLE) return false;
    *max_pairs = mpg::gemm_max_resident_pairs(dtype);
    if (*max_pairs <= 0) return false;
    if (policy == MPGEMMFI_TILES_PAIR) return true;
    const long long tiles = (long long)((M + 255) / 256) * ((N + 255) / 256);
    return M > 128 && N > 128 && tiles >= *max_pairs / 2;
}

int check_common(int dtype, int M, int N, int K, const void *A, const void *Bt, const void *C)
{
    if (dtype != MPGEMMFI_FP16 && dtype != MPGEMMFI_BF16 && dtype != MPGEMMFI_TF32) return MPGEMMFI_ERR_DTYPE;
    if (M <= 0 || N <= 0 || K <= 0 || !A || !Bt || !C) return MPGEMMFI_ERR_ARG;
    if ((unsigned long long)M * (unsigned long long)N >= 0xFFFFFFFFull) return MPGEMMFI_ERR_ARG;
    const int es = mpg::esize_of(dtype);
    if (((uintptr_t)A & 15) || ((uintptr_t)Bt & 15) || ((uintptr_t)C & 3) || ((size_t)K * es) % 16) return MPGEMMFI_ERR_ALIGN;
    return MPGEMMFI_OK;
}

int run_gemm(int dtype, int M, int N, int K, const void *A, const void *Bt, void *C, const mpgemmfi_site *sites,
             int n_faults, int detect_mode, uint32_t *flags, cudaStream_t stream, const DeviceInfo &di,
             const uint32_t *exp_a = nullptr, const uint32_t *exp_bt = nullptr, const float *addend = nullptr,
             int out_fmt = MPGEMMFI_OUT_FP32)
{
    Range range("mpgemmfi: gemm");
    int max_pairs = 0;
    const bool pair = choose_pair(dtype, M, N, &max_pairs);
    const int bn = pair ? 256 : choose_bn(M, N, di.num_sms);
    const int tm = pair ? 256 : 128;
    CUtensorMap tm_a, tm_b;
    int rc = encode_operand_map(&tm_a, dtype, A, M, K, 128);
    if (rc) return rc;
    rc = encode_operand_map(&tm_b, dtype, Bt, N, K, pair ? 128 : bn);
    if (rc) return rc;

    mpg::GemmParams p;
    p.dtype = dtype; p.M = M; p.N = N; p.K = K;
    p.detect_mode = detect_mode; p.n_faults = n_faults;
    p.tiles_m = (M + tm - 1) / tm; p.tiles_n = (N + bn - 1) / bn;
    p.num_tiles = p.tiles_m * p.tiles_n;
    // the walkers' tiles of one round should cover about as many bytes of A as of Bt
    p.group_m = pair ? 8 : (bn == 256 ? 16 : (bn == 128 ? 12 : 8));
    if (p.group_m > p.tiles_m) p.group_m = p.tiles_m;
    const int ks = mpg::kstep_of(dtype);
    p.num_kt = (K + ks - 1) / ks;
    p.wpr = (N + 31) / 32;
    p.out_fmt = out_fmt;
    const int out_es = out_fmt == MPGEMMFI_OUT_FP32 ? 4 : 2;
    p.c_vec_ok = (((size_t)N * out_es) % 16 == 0) && (((uintptr_t)C & 15) == 0);
    CUtensorMap tm_c;
    memset(&tm_c, 0, sizeof(tm_c));
    if (p.c_vec_ok) {
        rc = out_fmt == MPGEMMFI_OUT_FP32 ? encode_output_map(&tm_c, static_cast<float *>(C), M, N)
                                          : encode_output_map16(&tm_c, C, out_fmt, M, N);
        if (rc) return rc;
    }
    p.A = A; p.Bt = Bt; p.C = static_cast<float *>(C); p.sites = sites; p.flags = flags;
    p.sites_inline = 0;
    memset(p.inline_sites, 0, sizeof(p.inline_sites));
    if (n_faults > 0) {
        // a table in host memory rides in the launch parameters
        cudaPointerAttributes at;
        const cudaError_t ea = cudaPointerGetAttributes(&at, sites);
        if (ea != cudaSuccess) return cuda_fail(ea);
        if (at.type == cudaMemoryTypeUnregistered || at.type == cudaMemoryTypeHost) {
            if (n_faults > mpg::GEMM_INLINE_SITES) return MPGEMMFI_ERR_ARG;
            memcpy(p.inline_sites, sites, (size_t)n_faults * sizeof(mpgemmfi_site));
            p.sites_inline = 1;
            p.sites = nullptr;
        }
    }
    p.exp_a = exp_a; p.exp_b = exp_bt;
    p.addend = addend;
    p.addend_vec_ok = (N % 4 == 0) && (((uintptr_t)addend & 15) == 0);
    p.log2_k = 0;
    while ((1 << p.log2_k) < K) ++p.log2_k;
    const int walkers = pair ? max_pairs : di.num_sms;
    p.epoch = 0; p.signals = nullptr; p.ready = nullptr;
    p.wait_limit_ns = (uint64_t)g_wait_limit_ms * 1000000ull;
    p.tag_skew = g_break_handover ? 4u : 0u;        // test hook: an expected part number that nobody writes
    mpg::choose_split_schedule(p, walkers, g_split_policy.load());
    int slot = -1;
    if (p.split_parts > 1 || flags) {
        // (the header and the site log of `flags` are cleared by the kernel itself)
        const cudaError_t es = mpg::gemm_slot_acquire(stream, &slot, &p.epoch, &p.signals, &p.ready);
        if (es != cudaSuccess) return cuda_fail(es);
    }
    const int grid = (p.num_tiles < walkers ? p.num_tiles : walkers) * (pair ? 2 : 1);
    cudaError_t e = mpg::launch_gemm(bn, pair, tm_a, tm_b, tm_c, p, grid, stream);
    if (e == cudaSuccess && slot >= 0) e = mpg::gemm_slot_release(slot, stream);
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

}  // namespace

extern "C" {

int mpgemmfi_gemm(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C,
                  const mpgemmfi_site *fault_sites, int n_faults, int detect_mode, uint32_t *flags_out,
                  mpgemmfi_stream stream)
{
    int rc = check_common(dtype, M, N, K, A, Bt, C);
    if (rc) return rc;
    if (n_faults < 0 || n_faults > MPGEMMFI_MAX_FAULTS || (n_faults > 0 && !fault_sites)) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT)) return MPGEMMFI_ERR_ARG;
    if (!flags_out && (n_faults > 0 || (detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK))) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)fault_sites & 15) || ((uintptr_t)flags_out & 15)) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    return run_gemm(dtype, M, N, K, A, Bt, C, fault_sites, n_faults, detect_mode, flags_out,
                    static_cast<cudaStream_t>(stream), di);
}

int mpgemmfi_gemm_ranged(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C,
                         const mpgemmfi_site *fault_sites, int n_faults, int detect_mode, uint32_t *flags_out,
                         const uint32_t *exp_a, const uint32_t *exp_bt, mpgemmfi_stream stream)
{
    int rc = check_common(dtype, M, N, K, A, Bt, C);
    if (rc) return rc;
    if (n_faults < 0 || n_faults > MPGEMMFI_MAX_FAULTS || (n_faults > 0 && !fault_sites)) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT | MPGEMMFI_OUTPUT_RANGE)) return MPGEMMFI_ERR_ARG;
    const int tech = detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK;
    if (detect_mode & MPGEMMFI_OUTPUT_RANGE) {
        if (tech != MPGEMMFI_DETECT_RANGE_MAX && tech != MPGEMMFI_DETECT_RANGE_FLIP) return MPGEMMFI_ERR_ARG;
        if (!exp_a || !exp_bt) return MPGEMMFI_ERR_ARG;
        if (((uintptr_t)exp_a & 3) || ((uintptr_t)exp_bt & 3)) return MPGEMMFI_ERR_ALIGN;
    }
    if (!flags_out && (n_faults > 0 || tech)) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)fault_sites & 15) || ((uintptr_t)flags_out & 15)) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    const bool ranged = (detect_mode & MPGEMMFI_OUTPUT_RANGE) != 0;
    return run_gemm(dtype, M, N, K, A, Bt, C, fault_sites, n_faults, detect_mode, flags_out,
                    static_cast<cudaStream_t>(stream), di, ranged ? exp_a : nullptr, ranged ? exp_bt : nullptr);
}

int mpgemmfi_gemm_addend(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in, float *D,
                         const mpgemmfi_site *fault_sites, int n_faults, int detect_mode, uint32_t *flags_out,
                         mpgemmfi_stream stream)
{
    int rc = check_common(dtype, M, N, K, A, Bt, D);
    if (rc) return rc;
    if (!C_in) return MPGEMMFI_ERR_ARG;
    if ((uintptr_t)C_in & 3) return MPGEMMFI_ERR_ALIGN;
    // in place (C_in == D) is fine: a tile's addend is read before anything of that tile is written;
    // any other overlap would let one tile's stores reach another tile's addend
    const uintptr_t c0 = (uintptr_t)C_in, d0 = (uintptr_t)D;
    const size_t bytes = (size_t)M * (size_t)N * sizeof(float);
    if (c0 != d0 && c0 < d0 + bytes && d0 < c0 + bytes) return MPGEMMFI_ERR_ARG;
    if (n_faults < 0 || n_faults > MPGEMMFI_MAX_FAULTS || (n_faults > 0 && !fault_sites)) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT)) return MPGEMMFI_ERR_ARG;
    if (!flags_out && (n_faults > 0 || (detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK))) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)fault_sites & 15) || ((uintptr_t)flags_out & 15)) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    return run_gemm(dtype, M, N, K, A, Bt, D, fault_sites, n_faults, detect_mode, flags_out,
                    static_cast<cudaStream_t>(stream), di, nullptr, nullptr, C_in);
}

int mpgemmfi_gemm_out16(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in, int out_format,
                        void *D16, const mpgemmfi_site *fault_sites, int n_faults, int detect_mode, uint32_t *flags_out,
                        mpgemmfi_stream stream)
{
    if (out_format != MPGEMMFI_OUT_FP16 && out_format != MPGEMMFI_OUT_BF16) return MPGEMMFI_ERR_DTYPE;
    if (dtype != MPGEMMFI_FP16 && dtype != MPGEMMFI_BF16 && dtype != MPGEMMFI_TF32) return MPGEMMFI_ERR_DTYPE;
    if (M <= 0 || N <= 0 || K <= 0 || !A || !Bt || !D16) return MPGEMMFI_ERR_ARG;
    if ((unsigned long long)M * (unsigned long long)N >= 0xFFFFFFFFull) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)A & 15) || ((uintptr_t)Bt & 15) || ((uintptr_t)D16 & 1) || ((uintptr_t)C_in & 3) ||
        ((size_t)K * mpg::esize_of(dtype)) % 16)
        return MPGEMMFI_ERR_ALIGN;
    if (C_in) {
        // the addend is read tile by tile while other tiles' results are written: the two must not share memory
        const uintptr_t c0 = (uintptr_t)C_in, d0 = (uintptr_t)D16;
        if (c0 < d0 + (size_t)M * N * 2 && d0 < c0 + (size_t)M * N * 4) return MPGEMMFI_ERR_ARG;
    }
    if (n_faults < 0 || n_faults > MPGEMMFI_MAX_FAULTS || (n_faults > 0 && !fault_sites)) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT)) return MPGEMMFI_ERR_ARG;
    if (!flags_out && (n_faults > 0 || (detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK))) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)fault_sites & 15) || ((uintptr_t)flags_out & 15)) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    const int rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    return run_gemm(dtype, M, N, K, A, Bt, D16, fault_sites, n_faults, detect_mode, flags_out,
                    static_cast<cudaStream_t>(stream), di, nullptr, nullptr, C_in, out_format);
}

int mpgemmfi_operand_exponents(int dtype, int rows, int K, const void *X, uint32_t *out, mpgemmfi_stream stream)
{
    if (dtype != MPGEMMFI_FP16 && dtype != MPGEMMFI_BF16 && dtype != MPGEMMFI_TF32) return MPGEMMFI_ERR_DTYPE;
    if (rows <= 0 || K <= 0 || !X || !out) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)X & 15) || ((uintptr_t)out & 3) || ((size_t)K * mpg::esize_of(dtype)) % 16) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    const int rc = device_info(di);
    if (rc) return rc;
    const cudaError_t e = mpg::launch_operand_exponents(dtype, rows, K, X, out, di.num_sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

int mpgemmfi_campaign(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C_clean,
                      const mpgemmfi_site *sites, int n_trials, int detect_mode, mpgemmfi_trial_record *records,
                      void *workspace, size_t workspace_bytes, mpgemmfi_stream stream)
{
    int rc = check_common(dtype, M, N, K, A, Bt, C_clean);
    if (rc) return rc;
    if (n_trials < 0 || (n_trials > 0 && (!sites || !records))) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT | MPGEMMFI_TERM_HMMA_STEP | MPGEMMFI_TERM_IN_FORMAT)) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)sites & 15) || ((uintptr_t)records & 7)) return MPGEMMFI_ERR_ALIGN;
    if (!workspace || ((uintptr_t)workspace & 255) ||
        workspace_bytes < mpgemmfi_campaign_workspace_bytes(dtype, M, N, K, n_trials))
        return MPGEMMFI_ERR_WORKSPACE;
    DeviceInfo di;
    rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the clean product, shared by every trial
    rc = run_gemm(dtype, M, N, K, A, Bt, C_clean, nullptr, 0, MPGEMMFI_DETECT_NONE, nullptr, st, di);
    if (rc) return rc;
    mpg::CampaignParams p;
    p.dtype = dtype; p.M = M; p.N = N; p.K = K; p.detect_mode = detect_mode; p.n_trials = n_trials;
    p.A = A; p.Bt = Bt; p.C = C_clean; p.sites = sites; p.records = records;
    mpg::campaign_bind_schedule(p, workspace);
    Range range("mpgemmfi: campaign trials");
    const cudaError_t e = mpg::launch_campaign_trials(p, di.num_sms, st);
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

int mpgemmfi_campaign_static(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C_clean,
                             const mpgemmfi_site *sites, int n_trials, int detect_mode,
                             mpgemmfi_trial_record *records, mpgemmfi_stream stream)
{
    int rc = check_common(dtype, M, N, K, A, Bt, C_clean);
    if (rc) return rc;
    if (n_trials < 0 || (n_trials > 0 && (!sites || !records))) return MPGEMMFI_ERR_ARG;
    if (detect_mode & ~(MPGEMMFI_DETECT_TECHNIQUE_MASK | MPGEMMFI_CORRECT | MPGEMMFI_TERM_HMMA_STEP | MPGEMMFI_TERM_IN_FORMAT)) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)sites & 15) || ((uintptr_t)records & 7)) return MPGEMMFI_ERR_ALIGN;
    if (n_trials > MPGEMMFI_STATIC_MAX_TRIALS) return MPGEMMFI_ERR_WORKSPACE;   // built-in scratch too small
    DeviceInfo di;
    rc = device_info(di);
    if (rc) return rc;
    if (di.major != 10) return MPGEMMFI_ERR_ARCH;
    void *scratch = nullptr;
    size_t scratch_bytes = 0;
    cudaError_t e = mpg::campaign_static_schedule(&scratch, &scratch_bytes);
    if (e != cudaSuccess) return cuda_fail(e);
    if (scratch_bytes < mpg::campaign_schedule_bytes(n_trials)) return MPGEMMFI_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    rc = run_gemm(dtype, M, N, K, A, Bt, C_clean, nullptr, 0, MPGEMMFI_DETECT_NONE, nullptr, st, di);
    if (rc) return rc;
    mpg::CampaignParams p;
    p.dtype = dtype; p.M = M; p.N = N; p.K = K; p.detect_mode = detect_mode; p.n_trials = n_trials;
    p.A = A; p.Bt = Bt; p.C = C_clean; p.sites = sites; p.records = records;
    mpg::campaign_bind_schedule(p, scratch);
    Range range("mpgemmfi: campaign trials");
    e = mpg::launch_campaign_trials(p, di.num_sms, st);   // clears the schedule counters first
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

int mpgemmfi_campaign_summary(const mpgemmfi_trial_record *records, int n_trials, mpgemmfi_summary *summary,
                              mpgemmfi_stream stream)
{
    if (n_trials < 0 || (n_trials > 0 && !records) || !summary) return MPGEMMFI_ERR_ARG;
    if (((uintptr_t)records & 7) || ((uintptr_t)summary & 3)) return MPGEMMFI_ERR_ALIGN;
    DeviceInfo di;
    const int rc = device_info(di);
    if (rc) return rc;
    const cudaError_t e = mpg::launch_campaign_summary(records, n_trials, summary, di.num_sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

int mpgemmfi_set_tile_policy(int policy)
{
    if (policy != MPGEMMFI_TILES_AUTO && policy != MPGEMMFI_TILES_SINGLE && policy != MPGEMMFI_TILES_PAIR)
        return MPGEMMFI_ERR_ARG;
    g_tile_policy = policy;
    return MPGEMMFI_OK;
}

int mpgemmfi_set_split_policy(int policy)
{
    if (policy != MPGEMMFI_SPLIT_AUTO && policy != MPGEMMFI_SPLIT_OFF && policy != MPGEMMFI_SPLIT_ON)
        return MPGEMMFI_ERR_ARG;
    g_split_policy = policy;
    return MPGEMMFI_OK;
}

int mpgemmfi_set_wait_limit_ms(int ms)
{
    if (ms < 1 || ms > 60000) return MPGEMMFI_ERR_ARG;
    g_wait_limit_ms = ms;
    return MPGEMMFI_OK;
}

int mpgemmfi_debug_break_handover(int on)
{
    g_break_handover = on ? 1 : 0;
    return MPGEMMFI_OK;
}

int mpgemmfi_null_launch(mpgemmfi_stream stream)
{
    const cudaError_t e = mpg::launch_null(static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? MPGEMMFI_OK : cuda_fail(e);
}

int mpgemmfi_debug_launch_slot(uint32_t counter, uint32_t *epoch)
{
    if (epoch) *epoch = mpg::gemm_epoch_of(counter);
    return mpg::gemm_slot_of(counter);
}

int mpgemmfi_debug_segments(int num_tiles, int num_kt, int walkers, int policy, uint32_t *out, int max_out)
{
    if (num_tiles <= 0 || num_kt <= 0 || walkers <= 0 || max_out < 0 || (max_out > 0 && !out)) return MPGEMMFI_ERR_ARG;
    mpg::GemmParams p = {};
    p.num_tiles = num_tiles; p.num_kt = num_kt; p.c_vec_ok = 1; p.out_fmt = MPGEMMFI_OUT_FP32;
    mpg::choose_split_schedule(p, walkers, policy);
    const uint32_t groups = (uint32_t)(num_tiles < walkers ? num_tiles : walkers);
    int n = 0;
    for (uint32_t gid = 0; gid < groups; ++gid) {
        mpg::Segment sg;
        for (uint32_t i = 0; mpg::get_segment(p, gid, groups, i, sg); ++i, ++n) {
            if (n < max_out) {
                uint32_t *o = out + 8 * (size_t)n;
                o[0] = gid; o[1] = i; o[2] = sg.tile; o[3] = sg.kt0; o[4] = sg.kt1; o[5] = sg.part;
                o[6] = sg.load ? 1u : 0u; o[7] = sg.save ? 1u : 0u;
            }
        }
    }
    return n;
}

int mpgemmfi_kstep(int dtype)
{
    if (dtype != MPGEMMFI_FP16 && dtype != MPGEMMFI_BF16 && dtype != MPGEMMFI_TF32) return 0;
    return mpg::kstep_of(dtype);
}

size_t mpgemmfi_flags_bitmap_offset(int n_faults)
{
    return MPGEMMFI_HEADER_WORDS + 4 * (size_t)(n_faults > 0 ? n_faults : 0);
}

size_t mpgemmfi_flags_bytes(int M, int N, int n_faults)
{
    if (M <= 0 || N <= 0) return 0;
    return sizeof(uint32_t) * (mpgemmfi_flags_bitmap_offset(n_faults) + (size_t)M * (size_t)((N + 31) / 32));
}

size_t mpgemmfi_campaign_workspace_bytes(int dtype, int M, int N, int K, int n_trials)
{
    (void)dtype; (void)M; (void)N; (void)K;
    return mpg::campaign_schedule_bytes(n_trials);
}

int mpgemmfi_validate_sites(const mpgemmfi_site *host_sites, int n, int dtype, int M, int N, int K, int *first_bad)
{
    if (dtype != MPGEMMFI_FP16 && dtype != MPGEMMFI_BF16 && dtype != MPGEMMFI_TF32) return MPGEMMFI_ERR_DTYPE;
    if (n < 0 || (n > 0 && !host_sites) || M <= 0 || N <= 0 || K <= 0) return MPGEMMFI_ERR_ARG;
    for (int i = 0; i < n; ++i)
        if (!mpg::site_valid(host_sites[i], dtype, M, N, K)) {
            if (first_bad) *first_bad = i;
            return MPGEMMFI_ERR_SITE;
        }
    return MPGEMMFI_OK;
}

const char *mpgemmfi_strerror(int code)
{
    switch (code) {
    case MPGEMMFI_OK: return "ok";
    case MPGEMMFI_ERR_ARG: return "invalid argument";
    case MPGEMMFI_ERR_DTYPE: return "unknown dtype";
    case MPGEMMFI_ERR_ALIGN: return "pointer or row pitch not 16-byte aligned";
    case MPGEMMFI_ERR_SITE: return "fault site out of range";
    case MPGEMMFI_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case MPGEMMFI_ERR_ARCH: return "device is not sm_100";
    case MPGEMMFI_ERR_CUDA: return "CUDA call failed";
    default: return "unknown error";
    }
}

int mpgemmfi_last_cuda_error(void) { return g_last_cuda_error; }

int mpgemmfi_version(void) { return 100; }

}  // extern "C"
