/*
 * mpgemmfi -- fault-injected mixed-precision GEMM with in-kernel exponent-only
 * detection/correction, for NVIDIA B200 (sm_100a).
 *
 * C ABI. Every matrix pointer is a caller-owned DEVICE pointer that must stay
 * valid until the work queued on `stream` has completed. All entry points are
 * asynchronous and stream-ordered; none of them synchronises, and none allocates
 * device memory. Return value: MPGEMMFI_OK (0) or a negative MPGEMMFI_ERR_*.
 * Problems found on the device (a site outside the matrices, a wait that ran into
 * its time limit) never trap: they set bits in the status word of the flags header
 * (or the trial record) and the offending site is skipped.
 * A GEMM launch that has a flags buffer, or whose last round of tiles is cut (see
 * mpgemmfi_set_split_policy), carries a tag drawn from a counter when the entry point is
 * called, and uses one of 16 slots of a 160 KB static device array for the words its CTAs
 * hand to each other. Launches on several streams may overlap. A slot comes round again
 * every 16 such launches; the seventeenth is made to wait, on the device and in stream
 * order (an event per slot, no host synchronisation), until the launch that last held
 * its slot has finished, so any number of launches may be queued. A launch recorded once
 * and replayed (a CUDA graph) would reuse its tag and is not supported.
 *
 * Operation (paper Section II-B, IV-C): D = A x B with A (M x K) and B (K x N) in a
 * low-precision format -- FP16 (1/5/10), BF16 (1/8/7) or TF32 (1/8/10 held in a
 * 32-bit word, Section II-A) -- products accumulated into FP32, FP32 output.
 *
 * Layouts: A is M x K row-major (K contiguous). B is passed K-major as Bt[N][K]
 * (row j of Bt is column j of B). C is M x N row-major FP32. FP16/BF16 elements
 * are 2 bytes, TF32 elements are 4-byte FP32 words of which only the top 19 bits count
 * (the low 13 bits are ignored: truncated, not rounded).
 * A and Bt must be 16-byte aligned and K * element_size a multiple of 16 bytes.
 */
#ifndef MPGEMMFI_H
#define MPGEMMFI_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* `stream` is a cudaStream_t passed as an opaque pointer (NULL = default stream). */
typedef void *mpgemmfi_stream;

enum {
    MPGEMMFI_FP16 = 0,
    MPGEMMFI_BF16 = 1,
    MPGEMMFI_TF32 = 2
};

/*
 * Fault-site kinds. The paper's own fault is MPGEMMFI_SITE_TERM: bit flips in the
 * result of one multiplication, carried into the running sum by the write-back
 * of Eq. 1-2 (Section III-E, Section IV-A/IV-C). The other kinds place the same
 * XOR on an operand element, on a running accumulator, or on an output element.
 */
enum {
    MPGEMMFI_SITE_A = 0,    /* operand A[row, k]: storage bits ^= mask before the multiply   */
    MPGEMMFI_SITE_B = 1,    /* operand B[k, col] (= Bt[col, k])                               */
    MPGEMMFI_SITE_ACC = 2,  /* accumulator of C[row, col] after k elements were accumulated   */
    MPGEMMFI_SITE_OUT = 3,  /* output element C[row, col] before the output check             */
    MPGEMMFI_SITE_TERM = 4  /* product a[row,k]*b[k,col]: p' = p ^ mask; acc = (acc - p) + p' */
};

/*
 * One entry of the fault-site descriptor table (32 bytes).
 *   A / B : xor_mask addresses the operand's storage bits: bits 0..15 for FP16 and
 *           BF16; for TF32 mask bit b (0..18) addresses bit b+13 of the FP32 word.
 *   ACC   : k = number of k elements accumulated before the flip; must be a multiple
 *           of mpgemmfi_kstep(dtype), or equal to K; 0 < k <= K. 32-bit mask.
 *   TERM  : k = index of the term; the write-back is applied at the accumulator
 *           boundary that ends the k-step containing k. If a product-level check is
 *           selected it is applied to p' first (Section VI-B). 32-bit mask.
 *   OUT   : 32-bit mask on the FP32 output word.
 * Sites are applied in table order. `trial` is carried through for the caller.
 */
typedef struct {
    uint32_t kind;
    uint32_t row;
    uint32_t col;
    uint32_t k;
    uint32_t xor_mask;
    uint32_t trial;
    uint32_t pad[2];
} mpgemmfi_site;

/*
 * detect_mode: bits 1:0 select the technique (Section VI-A), bit 4 enables the
 * correction (applied only where the detection fires, Section VI-B).
 *   BOUNDCHECK : exponent MSB = 1 together with any of the next three exponent bits
 *                ("1eeexxxx", some e = 1, i.e. |v| >= 131072, Table III); correction
 *                clears the three e bits. Applied to TERM products and to every
 *                output element; only this technique produces output flags.
 *   RANGE_MAX  : faulty product exponent > e1 + e2 + 1; correction replaces it by
 *                that bound. Applied to TERM products only.
 *   RANGE_FLIP : same detection; correction clears the 1s of the exponent from its
 *                rightmost bit until it is <= the bound. TERM products only.
 */
enum {
    MPGEMMFI_DETECT_NONE = 0,
    MPGEMMFI_DETECT_BOUNDCHECK = 1,
    MPGEMMFI_DETECT_RANGE_MAX = 2,
    MPGEMMFI_DETECT_RANGE_FLIP = 3,
    MPGEMMFI_DETECT_TECHNIQUE_MASK = 3,
    MPGEMMFI_CORRECT = 16,
    /*
     * Campaigns only (mpgemmfi_gemm rejects it): a TERM trial's write-back takes place at the end
     * of the group of 16 (FP16, BF16) or 8 (TF32) terms that contains the term, i.e. on the
     * running sum as one HMMA instruction of the paper's platform leaves it (Section III-C:
     * shapes 16x8x16 and 16x8x8; Section IV-A: 16 or 8 terms per destination register), instead
     * of at the next mpgemmfi_kstep boundary.
     */
    MPGEMMFI_TERM_HMMA_STEP = 32,
    /*
     * Campaigns only: an alternative reading of where the paper's fault lands. Section IV-C flips bits "within the
     * result of a multiplication" without saying in which format that result is held; Section V-B's example of a
     * flipped zero is a 16-bit FP16 pattern, and the paper's format-dependent findings (Table II) need the product
     * to live in the operand format. With this flag a TERM trial rounds the product to the operand format (to
     * nearest even), applies xor_mask to that format's storage bits exactly as for an operand site (bits 0..15;
     * TF32: bits 0..18 addressing bits 13..31 of the word), widens the result back to FP32, and applies Eq. 1-2
     * with the rounded product as the term taken out and the flipped one as the term put in. The record's
     * before_bits / after_bits are then words of the operand format. Without the flag (the default, and what
     * mpgemmfi_gemm does) the flipped word is the FP32 product.
     */
    MPGEMMFI_TERM_IN_FORMAT = 128,
    /*
     * mpgemmfi_gemm_ranged only, together with RANGE_MAX or RANGE_FLIP: also range-check every
     * OUTPUT element. This extends the product bound of Section VI-A to a dot product and is not in
     * the paper: with EA_i / EB_j the largest FP32 exponent fields in row i of A / row j of Bt,
     * |C_ij| < K * 2^(eA+1) * 2^(eB+1), so the exponent field of C_ij is at most
     * EA_i + EB_j - 126 + ceil(log2 K) (clamped to 0..255). Detection: exponent above that bound;
     * correction as the technique says (replace by the bound / clear low exponent bits). The
     * maxima are taken over the CLEAN operands, so a faulty operand shows up in its row or column.
     */
    MPGEMMFI_OUTPUT_RANGE = 64
};

enum {
    MPGEMMFI_OK = 0,
    MPGEMMFI_ERR_ARG = -1,        /* null pointer, non-positive size, n_faults out of range */
    MPGEMMFI_ERR_DTYPE = -2,
    MPGEMMFI_ERR_ALIGN = -3,      /* pointer or row pitch not 16-byte aligned */
    MPGEMMFI_ERR_SITE = -4,       /* mpgemmfi_validate_sites: a site is out of range */
    MPGEMMFI_ERR_WORKSPACE = -5,  /* workspace too small or misaligned */
    MPGEMMFI_ERR_ARCH = -6,       /* current device is not sm_100 */
    MPGEMMFI_ERR_CUDA = -7        /* a CUDA runtime/driver call failed; see mpgemmfi_last_cuda_error() */
};

#define MPGEMMFI_MAX_FAULTS 4096      /* sites per mpgemmfi_gemm call */
#define MPGEMMFI_INLINE_FAULTS 8      /* sites a table in HOST memory may hold (it travels in the launch parameters) */
#define MPGEMMFI_HEADER_WORDS 16

/* status word of the flags header */
#define MPGEMMFI_STATUS_SITE_SKIPPED 1u  /* at least one site was invalid and skipped */
#define MPGEMMFI_STATUS_WAIT_LIMIT 2u    /* a device-side wait ran into its time limit; results invalid */

/*
 * flags_out layout (uint32 words):
 *   [0 .. 16)            header: [0] status, [1] n_detected, [2] n_corrected,
 *                        [3] sites applied, [4] sites skipped, [5] number of runs of k-steps the
 *                        tiles of the last round were cut into (0: whole tiles, see
 *                        mpgemmfi_set_split_policy), rest reserved (0)
 *   [16 .. 16+4*n_faults) site log, one entry per table entry (the paper logs the sum
 *                        before and after injection the same way, Section V-B):
 *                        {before_bits, after_bits, final_bits, status}
 *                          A/B : operand storage word before / after the XOR, final = after
 *                          ACC : accumulator bits before / after, final = after
 *                          TERM: product bits before / after the XOR, final = after the
 *                                product-level check; status bit 2 = detected
 *                          OUT : output bits before / after, final = after the output check
 *                        status: 1 applied, 2 skipped (invalid), bit 2 detected (TERM)
 *   [16+4*n_faults ..)   bitmap, M rows of ceil(N/32) words: bit (j mod 32) of word
 *                        i*ceil(N/32) + j/32 is 1 iff C[i,j] was detected (and corrected
 *                        when correction is on). Bits beyond column N-1 are 0.
 */
typedef struct {
    uint32_t before_bits;
    uint32_t after_bits;
    uint32_t final_bits;
    uint32_t status;
} mpgemmfi_site_log;

/*
 * One record per campaign trial (48 bytes). A trial is one site applied alone to
 * the clean GEMM (one fault per trial, Section IV-A).
 *   status        bit0 changed (some affected element's final bits differ from the
 *                 clean ones: the complement of the paper's "zero difference",
 *                 Section V-B), bit1 detected, bit2 corrected, bit8 invalid site
 *   primary_index OUT/ACC/TERM: row*N+col; A: row*K+k; B: col*K+k
 *   before/after  the word the mask was applied to, before and after the XOR
 *   final_bits    OUT/ACC/TERM: the output element after the check; A/B: = after_bits
 *   n_affected    output elements re-evaluated (1, N for an A site, M for a B site)
 *   n_detected    how many of them the output check flagged
 *   idx_hash      sum over flagged elements of (row*N+col+1) * 0x9E3779B97F4A7C15 mod 2^64
 *   first_detected smallest flagged row*N+col, 0xFFFFFFFF if none
 *   max_abs_dev   max over affected elements of |final - clean| (FP32; NaN counts as +inf)
 */
typedef struct {
    uint32_t status;
    uint32_t kind;
    uint32_t primary_index;
    uint32_t before_bits;
    uint32_t after_bits;
    uint32_t final_bits;
    uint32_t n_affected;
    uint32_t n_detected;
    uint64_t idx_hash;
    uint32_t first_detected;
    float max_abs_dev;
} mpgemmfi_trial_record;

/*
 * Fault-injected GEMM with the fused check (Sections II-B, III-E, IV-C, VI-A).
 *   A, Bt, C     device pointers, layouts above; C is written in full.
 *   fault_sites  device pointer to n_faults entries (may be NULL when n_faults = 0);
 *                0 <= n_faults <= MPGEMMFI_MAX_FAULTS.
 *                Alternatively a pointer to ordinary or pinned HOST memory holding at most
 *                MPGEMMFI_INLINE_FAULTS entries (the single fault of one trial, Section IV-A): the
 *                entries are copied during the call and travel in the kernel's launch parameters,
 *                so the caller may reuse the memory at once and the kernel reads no table from
 *                device memory (a table that is cold in the caches delays every CTA's start by
 *                a few microseconds). Which kind a pointer is, is asked of the CUDA runtime;
 *                managed memory counts as device memory. A host table with more entries: ERR_ARG.
 *                Results are identical either way. The same holds for every mpgemmfi_gemm_* below.
 *                The call is tuned for short tables (the paper's one fault per run): the time grows
 *                roughly linearly up to about 64 entries and faster beyond (a 4096^3 GEMM: 0.1 ms
 *                with one site, 0.13 ms with 64 operand sites, 0.6 ms with 1024); many independent
 *                faults are the business of mpgemmfi_campaign.
 *   flags_out    device pointer to mpgemmfi_flags_bytes(M, N, n_faults) bytes, 16-byte
 *                aligned, written in full; may be NULL only when n_faults = 0 and the
 *                technique is NONE (plain GEMM, nothing to report).
 * Errors: ERR_ARG, ERR_DTYPE, ERR_ALIGN, ERR_ARCH, ERR_CUDA.
 */
int mpgemmfi_gemm(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C,
                  const mpgemmfi_site *fault_sites, int n_faults, int detect_mode,
                  uint32_t *flags_out, mpgemmfi_stream stream);

/*
 * The same with an addend: D = A x B + C_in, the form the paper states the tensor-core operation in
 * (Section II-B). C_in is the accumulator the products are added to: every running sum starts from
 * c_in[i,j] instead of +0, so an ACC site at boundary k meets c_in[i,j] plus the first k products,
 * a TERM site's write-back (Eq. 1-2) acts on a sum that holds the addend, and OUT sites and the
 * output check see the finished d[i,j].
 *   C_in   device pointer, M x N FP32 row-major, 4-byte aligned (16-byte alignment and N a
 *          multiple of 4 let it be read 16 bytes at a time). It may be D itself (in place);
 *          any other overlap of the two matrices is refused with ERR_ARG.
 *   D      device pointer, M x N FP32 row-major, written in full.
 * Everything else as for mpgemmfi_gemm. Campaigns take no addend.
 */
int mpgemmfi_gemm_addend(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in,
                         float *D, const mpgemmfi_site *fault_sites, int n_faults, int detect_mode,
                         uint32_t *flags_out, mpgemmfi_stream stream);

/*
 * The same with a 16-bit result. The paper states the tensor-core operation as D = A x B + C with the
 * products accumulated in FP32 (Section II-B) and runs its models in "16" / "bf16" precision from end
 * to end (Section IV-B): the FP32 result of a layer's GEMM goes back to the 16-bit format before the
 * next layer reads it. Here everything up to and including the output check happens on the FP32 values
 * exactly as in mpgemmfi_gemm / mpgemmfi_gemm_addend (sites, flags, counts and the site log are those
 * of the FP32 result); then each element is rounded once, to nearest with ties to even, to
 * `out_format`: values beyond the format's range become infinities (FP16: |v| >= 65520), NaN stays
 * NaN (payload unspecified).
 *   C_in        NULL for D = A x B, or the FP32 addend (device, M x N, 4-byte aligned); it must not
 *               overlap D16 (ERR_ARG).
 *   out_format  MPGEMMFI_OUT_FP16 or MPGEMMFI_OUT_BF16 (ERR_DTYPE otherwise), independent of `dtype`.
 *   D16         device pointer, M x N row-major 2-byte words, written in full (16-byte alignment and
 *               N a multiple of 8 let it be written by bulk stores).
 * The last round of tiles is never cut for this entry point (see mpgemmfi_set_split_policy).
 * Everything else, and the errors, as for mpgemmfi_gemm.
 */
enum {
    MPGEMMFI_OUT_FP32 = 0,  /* what the other entry points write; not accepted here */
    MPGEMMFI_OUT_FP16 = 1,
    MPGEMMFI_OUT_BF16 = 2
};
int mpgemmfi_gemm_out16(int dtype, int M, int N, int K, const void *A, const void *Bt, const float *C_in,
                        int out_format, void *D16, const mpgemmfi_site *fault_sites, int n_faults,
                        int detect_mode, uint32_t *flags_out, mpgemmfi_stream stream);

/*
 * Largest FP32 exponent field of each row of a rows x K operand matrix (A, or Bt): out[r] in
 * 0..255; 0 for an all-zero row, 255 if the row holds Inf or NaN. X and out are device pointers
 * (X 16-byte aligned, K * element size a multiple of 16 bytes). Input of mpgemmfi_gemm_ranged.
 * No counterpart in the paper. Errors: ERR_ARG, ERR_DTYPE, ERR_ALIGN, ERR_CUDA.
 */
int mpgemmfi_operand_exponents(int dtype, int rows, int K, const void *X, uint32_t *out, mpgemmfi_stream stream);

/*
 * mpgemmfi_gemm with the output-level range check available: exp_a[M] and exp_bt[N] (device) are the
 * row maxima of the operands as mpgemmfi_operand_exponents gives them; they are only read when
 * detect_mode carries MPGEMMFI_OUTPUT_RANGE (and may be NULL otherwise). Everything else as
 * mpgemmfi_gemm, which itself rejects that flag.
 */
int mpgemmfi_gemm_ranged(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C,
                         const mpgemmfi_site *fault_sites, int n_faults, int detect_mode,
                         uint32_t *flags_out, const uint32_t *exp_a, const uint32_t *exp_bt,
                         mpgemmfi_stream stream);

/*
 * Injection campaign: ONE clean GEMM, then every trial is evaluated on the output
 * elements it can reach (Section IV-A: one fault per trial; Eq. 1-2 for how a
 * faulty term enters a finished sum).
 *   C_clean     device, M x N, written: the fault-free, unchecked product.
 *   sites       device, n_trials entries, one site per trial.
 *   records     device, n_trials records, written in full.
 *   workspace   device scratch of at least mpgemmfi_campaign_workspace_bytes(...)
 *               bytes, 256-byte aligned; contents undefined afterwards.
 * OUT trials flip the clean element. ACC and TERM trials recompute their element's
 * dot product in k order on the FP32 ALUs with the site active (and once without it,
 * which is the trial's clean reference). A and B trials apply, to every element of the
 * affected row or column, c' = (c - a*b) + a'*b with the clean and the faulty operand
 * (the write-back form of Eq. 1-2 applied to a finished sum). Every re-evaluated
 * element then goes through the output check of detect_mode.
 * Errors: as mpgemmfi_gemm, plus ERR_WORKSPACE.
 */
int mpgemmfi_campaign(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C_clean,
                      const mpgemmfi_site *sites, int n_trials, int detect_mode,
                      mpgemmfi_trial_record *records, void *workspace, size_t workspace_bytes,
                      mpgemmfi_stream stream);

/*
 * The campaign for callers that must not allocate device memory. (The paper has no
 * counterpart to this entry point; it exists for how the library gets embedded.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plugin or callback
 * invoked from inside someone else's pipeline, a real-time or long-running service that
 * froze its memory pools at start-up, or a host program whose device memory is handed
 * out by another owner. Such a caller has nowhere to get the `workspace` that
 * mpgemmfi_campaign asks for. Here the trial schedule lives instead in a fixed array
 * that is part of the library image: 256 + 12 * MPGEMMFI_STATIC_MAX_TRIALS bytes
 * (768.25 KiB) of device memory on every GPU that loads the library, held until the
 * process unloads it. The call itself allocates and frees nothing.
 *
 * Arguments, results and errors are those of mpgemmfi_campaign without `workspace` and
 * `workspace_bytes`; inputs, C_clean and records are still the caller's buffers.
 * n_trials above MPGEMMFI_STATIC_MAX_TRIALS is refused with MPGEMMFI_ERR_WORKSPACE
 * before anything is queued; split the table across several calls instead.
 *
 * The first call on each device looks up the array's device address (that device must be
 * current) and sets kernel attributes; make that first call outside any stream capture.
 * All calls on one device share the one array and it keeps whatever the previous call
 * left: each call clears the counters it needs on `stream` before use, so calls queued
 * one after another on a stream are safe, but two calls that can overlap on the GPU
 * (different streams, different host threads) race on it and corrupt each other's records.
 */
#define MPGEMMFI_STATIC_MAX_TRIALS 65536
int mpgemmfi_campaign_static(int dtype, int M, int N, int K, const void *A, const void *Bt, float *C_clean,
                             const mpgemmfi_site *sites, int n_trials, int detect_mode,
                             mpgemmfi_trial_record *records, mpgemmfi_stream stream);

/*
 * Numeric-deviation summary of a campaign (Section V-B: the share of trials whose sum did
 * not change, "zero difference" as in Table II, and the distribution of the non-zero
 * differences, which the paper plots as an ECDF on a log scale).
 *   dev_exponent_hist[e]  number of valid trials whose max_abs_dev is non-zero and has FP32
 *                         exponent field e: bin e covers [2^(e-127), 2^(e-126)); e = 0 holds
 *                         subnormal deviations, e = 255 infinite ones (NaN counts as infinite)
 *   kind_*[k]             the same counts split by site kind (index = MPGEMMFI_SITE_*)
 */
typedef struct {
    uint32_t n_trials;          /* records examined */
    uint32_t n_invalid;         /* records whose site was invalid (status bit 8); not counted below */
    uint32_t n_zero_diff;       /* status bit0 clear: every affected element kept its clean bits */
    uint32_t n_detected;        /* status bit1 */
    uint32_t n_corrected;       /* status bit2 */
    uint32_t n_nonfinite;       /* max_abs_dev infinite */
    uint32_t kind_trials[5];
    uint32_t kind_zero_diff[5];
    uint32_t dev_exponent_hist[256];
} mpgemmfi_summary;

/*
 * Reduce n_trials records (device) into *summary (device, 4-byte aligned, written in full).
 * Errors: ERR_ARG, ERR_ALIGN, ERR_CUDA.
 */
int mpgemmfi_campaign_summary(const mpgemmfi_trial_record *records, int n_trials, mpgemmfi_summary *summary,
                              mpgemmfi_stream stream);

/*
 * Tuning knob (no counterpart in the paper): how the GEMM kernel tiles the output.
 *   AUTO   the library decides from M and N (default)
 *   SINGLE every CTA computes whole 128 x {64,128,256} tiles
 *   PAIR   two CTAs on neighbouring SMs share one 256 x 256 tile and the Bt tile (tcgen05
 *          cta_group::2); falls back to SINGLE when the device cannot host such pairs
 * Process-wide; read once when a launch is queued (a host thread that changes it while another
 * queues a launch gives that launch the old or the new value). Results are the same fault
 * semantics either way; individual output values may differ in rounding between policies.
 * Returns MPGEMMFI_OK or MPGEMMFI_ERR_ARG.
 */
enum {
    MPGEMMFI_TILES_AUTO = 0,
    MPGEMMFI_TILES_SINGLE = 1,
    MPGEMMFI_TILES_PAIR = 2
};
int mpgemmfi_set_tile_policy(int policy);

/*
 * Tuning knob (no counterpart in the paper): what happens to the last round of tiles when the
 * tile count is not a multiple of the number of tile walkers (CTAs or CTA pairs), so that the last
 * round would leave walkers idle.
 *   AUTO   the library cuts that round's tiles along K when that shortens the launch (default)
 *   OFF    every tile is computed whole by one walker
 *   ON     cut whenever the shape allows it (more tiles than walkers, at most half as many tiles left
 *          over as walkers, C and N fit 16-byte accesses), also where it does not pay: for tests
 * A cut tile is run as two to four consecutive runs of k-steps by different walkers at different
 * times; the unfinished FP32 accumulators wait in the tile's place in C and go back into the
 * tensor core's accumulator memory before the next run, so every element is still one FP32
 * accumulation in increasing k, bit-identical to the uncut tile, and accumulator / term sites meet
 * the same running sum. While the launch runs, C therefore holds intermediate values in those
 * tiles. The hand-over between walkers uses 160 KB of static device memory of the library,
 * tagged per launch. Process-wide; read once when a launch is queued.
 * Returns MPGEMMFI_OK or MPGEMMFI_ERR_ARG.
 */
enum {
    MPGEMMFI_SPLIT_AUTO = 0,
    MPGEMMFI_SPLIT_OFF = 1,
    MPGEMMFI_SPLIT_ON = 2
};
int mpgemmfi_set_split_policy(int policy);

/*
 * Robustness knob (no counterpart in the paper): how long any single device-side wait of the GEMM
 * kernel (on a shared-memory barrier, on another CTA's hand-over of a cut tile, on the cleared
 * header) may last before the launch gives up. A launch that gives up frees its tensor memory,
 * returns normally and reports MPGEMMFI_STATUS_WAIT_LIMIT in the flags header; its C is invalid;
 * the device stays usable. ms in 1..60000, default 4000. Process-wide, read when a launch is
 * queued. Returns MPGEMMFI_OK or MPGEMMFI_ERR_ARG.
 */
int mpgemmfi_set_wait_limit_ms(int ms);

/*
 * Test hook (no counterpart in the paper): while on, the CTAs that continue a cut tile (see
 * mpgemmfi_set_split_policy) wait for a hand-over tag that nobody writes, so that their bounded
 * wait runs out and the give-up path above can be exercised without any fault. Launches queued
 * while it is on produce invalid results by design. Never switch it on outside a test.
 */
int mpgemmfi_debug_break_handover(int on);

/*
 * Measurement aid (no counterpart in the paper): queues a kernel of one thread that does nothing on
 * `stream`. Timed like a GEMM (event, launch, event) it gives what launching and completing any kernel
 * costs on the system by itself -- several microseconds, which is most of the time of a GEMM of one
 * wave of tiles and a few percent of a 4096^3 one. Errors: ERR_CUDA.
 */
int mpgemmfi_null_launch(mpgemmfi_stream stream);

/*
 * Host logic of the launch slots (no device needed): returns the slot (0..15) that the launch with
 * counter value `counter` uses and stores its tag (29 bits, never 0) in *tag (if non-NULL).
 */
int mpgemmfi_debug_launch_slot(uint32_t counter, uint32_t *tag);

/*
 * Host logic of the tile schedule (no device needed): for `num_tiles` output tiles of `num_kt` k-steps each on
 * `walkers` tile walkers (CTAs or CTA pairs) under split policy `policy`, writes one 8-word entry per piece of
 * work, walker by walker in the order the walker runs them: {walker, index, tile, first k-step, end k-step, part,
 * starts from the sums a previous part left in C (0/1), leaves its sums in C for the next part (0/1)}. At most
 * max_out entries are written; the return value is the number of entries there are (or MPGEMMFI_ERR_ARG). It assumes
 * an FP32 C that allows 16-byte accesses, as the split schedule requires.
 */
int mpgemmfi_debug_segments(int num_tiles, int num_kt, int walkers, int policy, uint32_t *out, int max_out);

/* k elements between two accumulator boundaries: 64 (FP16, BF16), 32 (TF32); 0 for a bad dtype. */
int mpgemmfi_kstep(int dtype);

/* bytes of the flags_out buffer for an M x N output and n_faults sites */
size_t mpgemmfi_flags_bytes(int M, int N, int n_faults);

/* offset, in uint32 words, of the bitmap inside flags_out */
size_t mpgemmfi_flags_bitmap_offset(int n_faults);

size_t mpgemmfi_campaign_workspace_bytes(int dtype, int M, int N, int K, int n_trials);

/*
 * Host-side check of a HOST copy of a site table: returns MPGEMMFI_OK, or
 * MPGEMMFI_ERR_SITE and stores the index of the first bad entry in *first_bad
 * (if non-NULL). The device applies the same rules and skips bad entries.
 */
int mpgemmfi_validate_sites(const mpgemmfi_site *host_sites, int n, int dtype, int M, int N, int K,
                            int *first_bad);

const char *mpgemmfi_strerror(int code);

/* cudaError_t value of the last failed CUDA call seen by this library (0 if none) */
int mpgemmfi_last_cuda_error(void);

/* major*10000 + minor*100 + patch */
int mpgemmfi_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MPGEMMFI_H */
