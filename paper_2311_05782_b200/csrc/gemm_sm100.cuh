// Host-visible interface of the tensor-core GEMM kernel.
#pragma once

#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/mpgemmfi.h"

namespace mpg {

// a site table of at most this many entries may travel in the launch parameters instead of device memory
constexpr int GEMM_INLINE_SITES = MPGEMMFI_INLINE_FAULTS;

struct GemmParams {
    int dtype, M, N, K;
    int detect_mode, n_faults;
    int tiles_m, tiles_n, num_tiles, num_kt;
    int group_m;    // tile rows per band of the tile order (>= 1)
    int wpr;        // bitmap words per row = ceil(N / 32)
    int c_vec_ok;   // C is 16-byte aligned with a 16-byte row pitch: the epilogue may use 16-byte stores
    int out_fmt;    // MPGEMMFI_OUT_FP32, or a 16-bit format: C then points to M x N 2-byte words
    const void *A;
    const void *Bt;
    float *C;
    const mpgemmfi_site *sites;     // the table in device memory; unused when sites_inline is set
    // The table given by value (n_faults <= GEMM_INLINE_SITES): the kernel then reads it from its parameters and
    // never waits for a (cold) line of device memory before its first operand copy.
    int sites_inline;
    mpgemmfi_site inline_sites[GEMM_INLINE_SITES];
    uint32_t *flags;
    // output-level range check (null when not requested): row exponent maxima of A and Bt, ceil(log2 K)
    const uint32_t *exp_a;
    const uint32_t *exp_b;
    int log2_k;
    // Addend of D = A x B + C (null: none): M x N FP32 that every tile's accumulators start from. It may be
    // the output itself (in place). addend_vec_ok: 16-byte aligned with a 16-byte row pitch.
    const float *addend;
    int addend_vec_ok;
    // Split schedule of the last round of tiles (split_parts <= 1: off). The tile walkers first share
    // out `full_rounds` whole tiles each; the `left_tiles` tiles that remain are cut along K into
    // `split_parts` parts run by different walkers, the accumulators travelling through C.
    int split_parts, full_rounds, left_tiles;
    uint32_t epoch;        // tag of this launch in the hand-over words and in *ready
    uint32_t *signals;     // SPLIT_SIGNAL_WORDS hand-over words of this launch (device memory)
    // With a flags buffer: CTA 0 clears the header and the site log when it starts, then stores `epoch`
    // here (release); any other CTA reads it (acquire, bounded wait) before it touches header or log.
    uint32_t *ready;
    // Every device-side wait (on a barrier, a hand-over word, *ready) gives up after this many nanoseconds; the
    // launch then ends with MPGEMMFI_STATUS_WAIT_LIMIT in the flags header instead of hanging.
    uint64_t wait_limit_ns;
    // XORed into the tag that the consumer of a cut tile waits for. Zero in every real launch; the tests set it so
    // that a hand-over never arrives and the give-up path runs.
    uint32_t tag_skew;
};

// One piece of work of a tile walker: k-tiles [kt0, kt1) of one output tile. `load`: the
// accumulators of k-tiles [0, kt0) come from C (left there by the walker of the previous part);
// `save`: the tile is not finished here, the raw accumulators go to C for the next part.
struct Segment {
    uint32_t tile, kt0, kt1, part;
    bool load, save;
};

// i-th segment of walker `gid`. Plain schedule (split_parts <= 1): tiles gid, gid + groups, ...,
// each whole. Split schedule: `full_rounds` whole tiles dealt out the same way, and the
// `left_tiles` tiles of the last round cut into `split_parts` equal runs of k-tiles; part g of
// left-over tile j belongs to walker g * left_tiles + j, which runs it after its g-th whole tile
// (the last part: after all of them), so that part g is finished long before part g + 1 starts.
__host__ __device__ inline bool get_segment(const GemmParams &p, uint32_t gid, uint32_t groups, uint32_t i, Segment &sg)
{
    const uint32_t nkt = (uint32_t)p.num_kt;
    if (p.split_parts <= 1) {
        sg.tile = gid + i * groups;
        sg.kt0 = 0; sg.kt1 = nkt; sg.part = 0; sg.load = false; sg.save = false;
        return sg.tile < (uint32_t)p.num_tiles;
    }
    const uint32_t left = (uint32_t)p.left_tiles, parts = (uint32_t)p.split_parts, rounds = (uint32_t)p.full_rounds;
    const uint32_t g = gid / left;
    const bool has_part = g < parts;
    const uint32_t pos = g + 1 < parts ? g : rounds;
    if (i >= rounds + (has_part ? 1u : 0u)) return false;
    if (has_part && i == pos) {
        sg.tile = groups * rounds + gid % left;
        sg.kt0 = g * nkt / parts; sg.kt1 = (g + 1) * nkt / parts; sg.part = g;
        sg.load = g > 0; sg.save = g + 1 < parts;
        return true;
    }
    sg.tile = gid + ((has_part && i > pos) ? i - 1 : i) * groups;
    sg.kt0 = 0; sg.kt1 = nkt; sg.part = 0; sg.load = false; sg.save = false;
    return true;
}

// hand-over words one launch can use: 16 per left-over tile, fewer left-over tiles than walkers
constexpr int SPLIT_MAX_WALKERS = 160;
constexpr int SPLIT_SIGNAL_WORDS = SPLIT_MAX_WALKERS * 16;

// Gives a launch its tag, its hand-over words and its ready word: a slot of a static device array,
// slots handed out in turn. A slot comes round again after LAUNCH_SLOTS launches; the tag keeps a
// launch from reading what an earlier one left there, and an event per slot keeps a launch from
// starting on a slot whose previous launch (on whatever stream) is still running:
// gemm_slot_acquire makes `stream` wait for that launch, gemm_slot_release (after the kernel has been
// queued on `stream`) records the slot's event there. The first acquire on a device creates the
// events. Both are cheap and never block the host.
constexpr int LAUNCH_SLOTS = 16;
constexpr int LAUNCH_SLOT_WORDS = SPLIT_SIGNAL_WORDS + 16;
cudaError_t gemm_slot_acquire(cudaStream_t stream, int *slot, uint32_t *epoch, uint32_t **signals, uint32_t **ready);
cudaError_t gemm_slot_release(int slot, cudaStream_t stream);
// slot index a launch counter value maps to (host logic, testable without a device)
inline int gemm_slot_of(uint32_t counter) { return (int)(counter % (uint32_t)LAUNCH_SLOTS); }
// 29-bit tag of a launch counter value, never 0 (three more bits carry a part number)
inline uint32_t gemm_epoch_of(uint32_t counter) { return (counter & 0x1FFFFFFFu) ? (counter & 0x1FFFFFFFu) : 1u; }

// Single mode (pair = false): bn in {64, 128, 256} is the width of the 128-row output tile; tm_b
// must have been encoded with a box of (128 bytes x bn rows); `grid` CTAs; p.tiles_m counts
// 128-row tiles.
// Pair mode (pair = true): 256 x 256 tiles walked by CTA pairs; tm_b box is (128 bytes x 128 rows);
// `grid` is even (two CTAs per pair); p.tiles_m counts 256-row tiles.
// tm_a always has a box of (128 bytes x 128 rows). Both maps use the 128-byte swizzle.
// tm_c covers C and is used for the stores of finished tiles when p.c_vec_ok is set (otherwise its contents do
// not matter): FP32 output: box 32 columns x 16 rows, 128-byte swizzle; 16-bit output: box 32 columns x 32 rows,
// 64-byte swizzle.
// Split schedule for `tiles` tiles of `num_kt` k-tiles on `walkers` tile walkers under `policy` (MPGEMMFI_SPLIT_*): fills
// split_parts / full_rounds / left_tiles of p (split_parts 0: every tile whole). Off unless there is at least one full
// round, the left-over tiles number at most half the walkers, every part keeps at least four k-tiles, C allows 16-byte
// accesses and is FP32, and (policy AUTO) the launch gets visibly shorter. Host logic, no device needed.
void choose_split_schedule(GemmParams &p, int walkers, int policy);

cudaError_t launch_gemm(int bn, bool pair, const CUtensorMap &tm_a, const CUtensorMap &tm_b, const CUtensorMap &tm_c,
                        const GemmParams &p, int grid, cudaStream_t stream);

// how many CTA pairs of the pair-mode kernel can be resident at once on the current device (0 if none)
int gemm_max_resident_pairs(int dtype);

}  // namespace mpg
