// Fault-injected mixed-precision GEMM for sm_100a.
//
// One persistent CTA per SM walks 128 x BN output tiles. Warp roles:
//   warp 0    TMA producer: k-tiles of A (128 rows x 128 bytes) and Bt (BN rows x 128 bytes)
//             into a ring of 128-byte-swizzled shared-memory stages
//   warp 1    MMA issuer: tcgen05.mma into one of two TMEM accumulators; flips operand
//             sites in the staged tiles before the tensor core reads them; pauses at the
//             k-step boundaries where an accumulator or product-term site takes effect
//   warp 2    TMEM allocation / release
//   warps 4-11 epilogue (warp w: TMEM lanes 32*(w%4).., left or right half of the tile's columns):
//             TMEM -> registers, accumulator / term write-back sites at the paused boundaries,
//             output-site flips, BoundCheck flags (+ correction), stores
//
// The fault-site table is decoded once per CTA into a list of the entries that touch any of
// its tiles; a CTA whose list is empty never looks at a site again.
//
// Two launch shapes share this code. Single: every CTA owns whole 128 x BN tiles. Pair: two
// CTAs (a cluster of two on neighbouring SMs) own one 256 x 256 tile; each stages its own 128
// rows of A and its own 128-row half of Bt, the leader CTA issues cta_group::2 MMAs that read
// both CTAs' shared memory and fill both CTAs' TMEM, and each CTA runs the epilogue of its own
// 128 rows. Halving the Bt bytes each SM has to pull per MMA is what lifts the main loop off
// the SM's shared-memory fill rate.
//
// Tile schedule. Tiles are dealt out round-robin to the tile walkers (CTAs or CTA pairs). When the
// last round would leave many walkers idle, its tiles are cut along K into parts that different
// walkers run at different times: the walker of part 0 runs it before its full tiles and leaves the
// raw accumulators in the tile's place in C; the walker of the last part runs after its full tiles,
// loads those accumulators back into TMEM and carries on with the next k-tile, so every element
// still sees one FP32 accumulation in increasing k, bit for bit the one of an uncut tile, and an
// accumulator site still meets the running sum. Parts in between sit after the walker's g-th full
// tile. A part's hand-over is one flag word per epilogue warp in a per-launch slot of a static
// device array; the waits on it are bounded like every other wait here.
#include <mutex>
#include <cstdint>
#include <type_traits>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "checks.cuh"
#include "gemm_sm100.cuh"
#include "ptx_sm100.cuh"

namespace mpg {

namespace {

constexpr uint32_t NONE = 0xFFFFFFFFu;
// check modes of the epilogue: none, BoundCheck (detect), BoundCheck + correction, output-level range check
enum { EPI_PLAIN = 0, EPI_BOUND = 1, EPI_BOUND_CORRECT = 2, EPI_RANGE = 3 };
constexpr int BM = 128;
constexpr int NUM_THREADS = 384;     // 4 control warps + 8 epilogue warps
constexpr int EPI_WARPS = 8;
constexpr int SITE_CACHE = 64;
constexpr int SINGLE_SITE_WARP = 3;       // the warp with no other role, see build_site_list
constexpr int MAX_STAGES = 8;
constexpr int OUT_BUF_BYTES = 16 * 128;                    // staging of one epilogue warp: 16 rows x 128 bytes
constexpr int OUT_STAGING_BYTES = EPI_WARPS * OUT_BUF_BYTES;
constexpr int SMEM_LIMIT = 227 * 1024;                    // dynamic shared memory one CTA may have
constexpr int CONTROL_RESERVE = 12 * 1024;                 // control block + 1 KB of alignment slack

template <int BN, bool kPair>
struct Cfg {
    static constexpr int B_ROWS = kPair ? BN / 2 : BN;     // Bt rows staged by one CTA
    static constexpr int A_BYTES = BM * 128;
    static constexpr int B_BYTES = B_ROWS * 128;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    // the operand ring gets what the output staging and the control block leave
    static constexpr int STAGES_FIT = (SMEM_LIMIT - CONTROL_RESERVE - OUT_STAGING_BYTES) / STAGE_BYTES;
    static constexpr int STAGES = STAGES_FIT < MAX_STAGES ? STAGES_FIT : MAX_STAGES;
    static_assert(STAGES >= 3, "operand ring too short");
    // (the last tile's epilogue parks 4 KB per 32-column piece in the ring: 8 warps x BN / 64 pieces each)
    static_assert(STAGES * STAGE_BYTES >= EPI_WARPS * (BN / 64) * 4096, "operand ring smaller than the last tile's staging");
    static constexpr int TMEM_COLS = 2 * BN;   // two accumulators; 128, 256 or 512 columns
    static_assert(BN == 64 || BN == 128 || BN == 256, "BN must be 64, 128 or 256");
    static_assert(!kPair || BN == 256, "pair tiles are 256 x 256");
};

// Control block that follows the stages in dynamic shared memory.
struct alignas(16) Control {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[2];
    uint64_t acc_empty[2];
    uint64_t pause_full;
    uint64_t pause_done;
    uint64_t acc_loaded[2];   // accumulator buffer s holds what its next segment starts from (a continued tile part, an addend)
    uint32_t tmem_base;
    uint32_t abort_flag;
    uint32_t site_count;
    uint32_t pad;
    // The CTA's list holds its sites by class, each class in table order: operand sites (A, B) in
    // [0, class_end[0]), accumulator and term sites in [class_end[0], class_end[1]), output sites in
    // [class_end[1], site_count): every role walks only the entries it can do something with.
    uint32_t class_end[2];
    uint32_t scan[3][NUM_THREADS / 32];
    uint16_t site_idx[MPGEMMFI_MAX_FAULTS];
    mpgemmfi_site site_cache[SITE_CACHE];     // the first entries of the CTA's list, so that scans stay on chip
};

// Ranges of one output tile as seen by one CTA. In single mode "own" and "tile" coincide; in pair
// mode the tile is 256 rows tall, the CTA owns 128 of them and a 128-row half of the Bt tile.
struct TileCtx {
    const GemmParams *p;
    const Control *ctl;
    uint32_t m0, n0;        // rows of C / A this CTA computes, first column of the tile
    uint32_t tile_m0;       // first row of the whole tile
    uint32_t b0;            // first Bt row (column of C) this CTA stages
    uint32_t tile_rows, bn, b_rows;
};

__device__ __forceinline__ bool in_own_rows(const TileCtx &c, uint32_t row) { return row - c.m0 < (uint32_t)BM; }
__device__ __forceinline__ bool in_tile_rows(const TileCtx &c, uint32_t row) { return row - c.tile_m0 < c.tile_rows; }
__device__ __forceinline__ bool in_tile_cols(const TileCtx &c, uint32_t col) { return col - c.n0 < c.bn; }
__device__ __forceinline__ bool in_own_b(const TileCtx &c, uint32_t col) { return col - c.b0 < c.b_rows; }

// entry i of the site table: from the launch parameters when the table travels there, else from device memory
__device__ __forceinline__ mpgemmfi_site table_site(const GemmParams &p, int i)
{
    if (p.sites_inline) return p.inline_sites[i & (GEMM_INLINE_SITES - 1)];
    return load_site(p.sites, i);
}

// class of a site kind in the CTA's list (see Control::class_end)
__device__ __forceinline__ int site_class(uint32_t kind)
{
    return (kind == MPGEMMFI_SITE_A || kind == MPGEMMFI_SITE_B) ? 0 : (kind == MPGEMMFI_SITE_OUT ? 2 : 1);
}

// entry i of the CTA's site list: from shared memory for the first SITE_CACHE entries
__device__ __forceinline__ mpgemmfi_site listed_site(const TileCtx &c, uint32_t i)
{
    if (i < (uint32_t)SITE_CACHE) return c.ctl->site_cache[i];
    return table_site(*c.p, c.ctl->site_idx[i]);
}

// smallest k-tile >= kt_from in which this tile has an operand site (warp-wide)
__device__ uint32_t scan_next_operand(const TileCtx &c, uint32_t kt_from, int lane)
{
    const uint32_t sh = kshift_of(c.p->dtype);
    if (c.ctl->site_count == 1) {          // the usual table: one site, no loop and no warp-wide reduction
        const mpgemmfi_site s = c.ctl->site_cache[0];
        const bool hit = (s.kind == MPGEMMFI_SITE_A && in_own_rows(c, s.row)) ||
                         (s.kind == MPGEMMFI_SITE_B && in_own_b(c, s.col));
        return (hit && (s.k >> sh) >= kt_from) ? s.k >> sh : NONE;
    }
    uint32_t best = NONE;
    for (uint32_t i = lane; i < c.ctl->class_end[0]; i += 32) {
        const mpgemmfi_site s = listed_site(c, i);
        const bool hit = (s.kind == MPGEMMFI_SITE_A && in_own_rows(c, s.row)) ||
                         (s.kind == MPGEMMFI_SITE_B && in_own_b(c, s.col));
        if (hit && (s.k >> sh) >= kt_from) best = min(best, s.k >> sh);
    }
    return __reduce_min_sync(0xFFFFFFFFu, best);
}

// smallest boundary >= b_from at which this tile has an accumulator / term site (warp-wide)
__device__ uint32_t scan_next_boundary(const TileCtx &c, uint32_t b_from, int lane)
{
    if (c.ctl->site_count == 1) {
        const mpgemmfi_site s = c.ctl->site_cache[0];
        if ((s.kind == MPGEMMFI_SITE_ACC || s.kind == MPGEMMFI_SITE_TERM) && in_tile_rows(c, s.row) && in_tile_cols(c, s.col)) {
            const uint32_t b = site_boundary(s, c.p->dtype, c.p->K);
            if (b >= b_from) return b;
        }
        return NONE;
    }
    uint32_t best = NONE;
    for (uint32_t i = c.ctl->class_end[0] + (uint32_t)lane; i < c.ctl->class_end[1]; i += 32) {
        const mpgemmfi_site s = listed_site(c, i);
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
    if (c.ctl->site_count == 1) {
        const mpgemmfi_site s = c.ctl->site_cache[0];
        return s.kind == MPGEMMFI_SITE_OUT && in_own_rows(c, s.row) && in_tile_cols(c, s.col);
    }
    bool any = false;
    for (uint32_t i = c.ctl->class_end[1] + (uint32_t)lane; i < c.ctl->site_count; i += 32) {
        const mpgemmfi_site s = listed_site(c, i);
        any |= s.kind == MPGEMMFI_SITE_OUT && in_own_rows(c, s.row) && in_tile_cols(c, s.col);
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

// One thread: XOR operand site `s` (entry `idx` of the table, known to lie in k-tile `kt` of this CTA's staged rows)
// into the staged tile and log it where this CTA is the one that reports the site.
__device__ __forceinline__ void flip_staged_operand(const TileCtx &c, const mpgemmfi_site &s, uint32_t idx, uint8_t *tile,
                                                    uint32_t r, bool log_here)
{
    const GemmParams &p = *c.p;
    const uint32_t sh = kshift_of(p.dtype);
    const uint32_t es = (uint32_t)esize_of(p.dtype);
    uint8_t *ptr = tile + swizzled_offset(r, (s.k & ((1u << sh) - 1u)) * es);
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

// which staged tile and row of it operand site s touches in k-tile kt of this CTA (tile == nullptr: none)
__device__ __forceinline__ void staged_place(const TileCtx &c, const mpgemmfi_site &s, uint32_t kt, uint8_t *smem_a, uint8_t *smem_b,
                                             uint8_t *&tile, uint32_t &r, bool &log_here)
{
    tile = nullptr; r = 0; log_here = false;
    if ((s.k >> kshift_of(c.p->dtype)) != kt) return;
    if (s.kind == MPGEMMFI_SITE_A && in_own_rows(c, s.row)) { tile = smem_a; r = s.row - c.m0; log_here = c.n0 == 0; }
    else if (s.kind == MPGEMMFI_SITE_B && in_own_b(c, s.col)) { tile = smem_b; r = s.col - c.b0; log_here = c.tile_m0 == 0; }
}

// The whole warp: XOR the operand sites of k-tile `kt` into the staged A / Bt tiles. A list of one entry (the usual
// case) is handled by lane 0 alone. Otherwise the lanes look through the operand entries of the CTA's list 32 at a
// time; the entries that hit this k-tile are applied one after the other in table order (two flips of one word log
// their before / after words in that order), each by the lane that holds it. A lane that has written fences its
// writes towards the tensor core's (asynchronous) reads.
__device__ __noinline__ void apply_operand_sites_many(TileCtx c, uint32_t kt, uint8_t *smem_a, uint8_t *smem_b, int lane);

__device__ __forceinline__ void apply_operand_sites(const TileCtx &c, uint32_t kt, uint8_t *smem_a, uint8_t *smem_b, int lane)
{
    uint8_t *tile;
    uint32_t r;
    bool log_here;
    if (c.ctl->site_count == 1) {
        if (lane == 0) {
            const mpgemmfi_site s = c.ctl->site_cache[0];
            staged_place(c, s, kt, smem_a, smem_b, tile, r, log_here);
            if (tile) { flip_staged_operand(c, s, c.ctl->site_idx[0], tile, r, log_here); fence_proxy_async_smem(); }
        }
        __syncwarp();
        return;
    }
    apply_operand_sites_many(c, kt, smem_a, smem_b, lane);
}

// (kept out of line, like the long form of build_site_list: the code of the one-site case stays short)
__device__ __noinline__ void apply_operand_sites_many(TileCtx c, uint32_t kt, uint8_t *smem_a, uint8_t *smem_b, int lane)
{
    uint8_t *tile;
    uint32_t r;
    bool log_here;
    const uint32_t n_op = c.ctl->class_end[0];
    for (uint32_t base = 0; base < n_op; base += 32) {
        const uint32_t i = base + (uint32_t)lane;
        mpgemmfi_site s = {};
        tile = nullptr; r = 0; log_here = false;
        if (i < n_op) {
            s = listed_site(c, i);
            staged_place(c, s, kt, smem_a, smem_b, tile, r, log_here);
        }
        uint32_t vote = __ballot_sync(0xFFFFFFFFu, tile != nullptr);
        while (vote) {
            const int turn = __ffs(vote) - 1;
            vote &= vote - 1u;
            if (lane == turn) {
                flip_staged_operand(c, s, c.ctl->site_idx[i], tile, r, log_here);
                fence_proxy_async_smem();
            }
            __syncwarp();
        }
    }
}

// operand word of A[row,k] or Bt[col,k] with every operand site of the table applied
__device__ uint32_t faulty_operand(const TileCtx &c, bool is_a, uint32_t rc, uint32_t k)
{
    const GemmParams &p = *c.p;
    uint32_t w = load_operand(p.dtype, is_a ? p.A : p.Bt, (size_t)rc * p.K + k);
    for (uint32_t i = 0; i < c.ctl->class_end[0]; ++i) {
        const mpgemmfi_site s = listed_site(c, i);
        if (s.k != k) continue;
        if (is_a ? (s.kind == MPGEMMFI_SITE_A && s.row == rc) : (s.kind == MPGEMMFI_SITE_B && s.col == rc))
            w = flip_operand(p.dtype, w, s.xor_mask);
    }
    return w;
}

// Epilogue warp of lane quarter q and column half h: apply, in table order, the accumulator and
// term sites of boundary b that live in its 32 TMEM lanes and its half of the columns.
__device__ void apply_boundary_sites(const TileCtx &c, uint32_t b, uint32_t tmem_acc, int q, int h, int lane)
{
    const GemmParams &p = *c.p;
    for (uint32_t i = c.ctl->class_end[0]; i < c.ctl->class_end[1]; ++i) {
        const uint32_t idx = c.ctl->site_idx[i];
        const mpgemmfi_site s = listed_site(c, i);
        if (!(s.kind == MPGEMMFI_SITE_ACC || s.kind == MPGEMMFI_SITE_TERM)) continue;
        if (!in_own_rows(c, s.row) || !in_tile_cols(c, s.col)) continue;
        if (site_boundary(s, p.dtype, p.K) != b) continue;
        const uint32_t r = s.row - c.m0;
        if ((int)(r >> 5) != q || (int)((s.col - c.n0) / (c.bn / 2)) != h) continue;
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

// Output sites of one thread's row inside the W-column piece starting at column c0.
// pass 0: XOR and log before/after; pass 1 (after the check): log the final bits.
template <int W>
__device__ void apply_out_sites(const TileCtx &c, uint32_t row, uint32_t c0, uint32_t (&v)[W], int pass)
{
    const GemmParams &p = *c.p;
    for (uint32_t i = c.ctl->class_end[1]; i < c.ctl->site_count; ++i) {
        const uint32_t idx = c.ctl->site_idx[i];
        const mpgemmfi_site s = listed_site(c, i);
        if (s.kind != MPGEMMFI_SITE_OUT || s.row != row || s.col - c0 >= (uint32_t)W) continue;
        const uint32_t j = s.col - c0;
#pragma unroll
        for (uint32_t jj = 0; jj < (uint32_t)W; ++jj) {
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

// Tile order. Tiles are numbered so that the tiles in flight at one time (consecutive numbers, dealt
// out round-robin to the walkers) form a block of group_m tile rows by several tile columns rather
// than one long column strip: each round then touches few row panels of A and few column panels of
// Bt, which keeps them in L2 when A or Bt alone is larger than L2.
// Within a band of group_m tile rows the number runs down the rows first, then across the columns.
__device__ __forceinline__ void tile_coords(const GemmParams &p, uint32_t t, uint32_t &tm, uint32_t &tn)
{
    const uint32_t band_tiles = (uint32_t)p.group_m * (uint32_t)p.tiles_n;
    const uint32_t band = t / band_tiles, within = t % band_tiles;
    const uint32_t rows = min((uint32_t)p.group_m, (uint32_t)p.tiles_m - band * (uint32_t)p.group_m);
    tm = band * (uint32_t)p.group_m + within % rows;
    tn = within / rows;
}

__device__ __forceinline__ uint32_t tile_number(const GemmParams &p, uint32_t tm, uint32_t tn)
{
    const uint32_t band = tm / (uint32_t)p.group_m;
    const uint32_t rows = min((uint32_t)p.group_m, (uint32_t)p.tiles_m - band * (uint32_t)p.group_m);
    return band * (uint32_t)p.group_m * (uint32_t)p.tiles_n + tn * rows + (tm - band * (uint32_t)p.group_m);
}

// Do the accumulators of this segment start from memory (the previous part's sums left in C, or the
// addend of D = A x B + C at a tile's first k-tile) rather than from the first MMA's overwrite?
__device__ __forceinline__ bool starts_from_memory(const GemmParams &p, const Segment &sg)
{
    return sg.load || (p.addend != nullptr && sg.kt0 == 0);
}

// does walker `gid` run tile t, whole or in part?
__device__ __forceinline__ bool walker_has_tile(const GemmParams &p, uint32_t t, uint32_t gid, uint32_t groups)
{
    if (p.split_parts > 1 && t >= groups * (uint32_t)p.full_rounds) {
        const uint32_t j = t - groups * (uint32_t)p.full_rounds;
        return gid % (uint32_t)p.left_tiles == j && gid / (uint32_t)p.left_tiles < (uint32_t)p.split_parts;
    }
    return t % groups == gid;
}

// Does a site touch a tile walked by tile-walker `gid` of `groups` (a CTA, or a CTA pair)?
// Tiles are TM x BN.
template <int TM, int BN>
__device__ bool site_touches_group(const mpgemmfi_site &s, const GemmParams &p, uint32_t gid, uint32_t groups)
{
    if (s.kind == MPGEMMFI_SITE_A) {
        const uint32_t tm = s.row / TM;
        for (uint32_t tn = 0; tn < (uint32_t)p.tiles_n; ++tn)
            if (walker_has_tile(p, tile_number(p, tm, tn), gid, groups)) return true;
        return false;
    }
    if (s.kind == MPGEMMFI_SITE_B) {
        const uint32_t tn = s.col / BN;
        for (uint32_t tm = 0; tm < (uint32_t)p.tiles_m; ++tm)
            if (walker_has_tile(p, tile_number(p, tm, tn), gid, groups)) return true;
        return false;
    }
    return walker_has_tile(p, tile_number(p, s.row / TM, s.col / BN), gid, groups);
}

// The same question asked by a whole warp about ONE site (the same `s` in every lane): the tiles of an operand
// site's row / column of tiles are shared out over the lanes, 32 per round, and a round with a hit ends the search.
// (One thread alone runs a division chain per tile: 3 us for the 16 tiles of a 4096-wide row, far more for the
// thousands of tile rows of a tall matrix.)
template <int TM, int BN>
__device__ bool site_touches_group_warp(const mpgemmfi_site &s, const GemmParams &p, uint32_t gid, uint32_t groups, int lane)
{
    if (s.kind == MPGEMMFI_SITE_A || s.kind == MPGEMMFI_SITE_B) {
        const bool is_a = s.kind == MPGEMMFI_SITE_A;
        const uint32_t fixed = is_a ? s.row / TM : s.col / BN;
        const uint32_t count = is_a ? (uint32_t)p.tiles_n : (uint32_t)p.tiles_m;
        for (uint32_t base = 0; base < count; base += 32) {
            const uint32_t i = base + (uint32_t)lane;
            const bool hit = i < count && walker_has_tile(p, is_a ? tile_number(p, fixed, i) : tile_number(p, i, fixed), gid, groups);
            if (__any_sync(0xFFFFFFFFu, hit)) return true;
        }
        return false;
    }
    return walker_has_tile(p, tile_number(p, s.row / TM, s.col / BN), gid, groups);
}

// Hand-over of a tile part between walkers: one word per epilogue warp of the walker.
__device__ __forceinline__ void signal_store_release(uint32_t *ptr, uint32_t v)
{
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(ptr), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t signal_load_acquire(const uint32_t *ptr)
{
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
    return v;
}

// bounded wait for *ptr == want; same give-up rules as mbar_wait
__device__ __forceinline__ bool signal_wait(const uint32_t *ptr, uint32_t want, volatile uint32_t *abort_flag,
                                            uint64_t limit_ns)
{
    if (signal_load_acquire(ptr) == want) return true;
    uint64_t t0 = 0;
    for (uint32_t it = 1;; ++it) {
        if (signal_load_acquire(ptr) == want) return true;
        __nanosleep(64);
        if ((it & 0x3Fu) == 0) {
            if (*abort_flag) return false;
            const uint64_t now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
        }
    }
}

// One epilogue warp, for a continued tile part that its walker runs later: wait for the warp of the
// previous part's walker that owns the same rows and columns (hand-over word *sig == want), then copy
// rows row0..row0+31, columns col0..col0+32*pieces-1 of the accumulators it left in C back into TMEM
// (this warp's lanes, columns from t_dst on). `park` is the warp's 2 KB of shared-memory staging.
// With sig == nullptr nothing is waited for (an addend: the caller's matrix is there already); with
// vec == false the source allows no 16-byte accesses and is read word by word.
// The store transpose of the epilogue run backwards: every load instruction reads whole 128-byte rows
// of C (lane l: 16-byte piece l % 8 of rows l / 8 + 4 it) and parks them in shared memory, then the
// threads of one half-warp pick up their own rows. (One 128-byte row per thread instead: 11 us per
// tile, during which the main loop next to it stood still.) Returns false when the wait gave up.
__device__ __forceinline__ bool load_partial(const float *C, uint32_t M, uint32_t N, const uint32_t *sig, uint32_t want,
                                             volatile uint32_t *abort_flag, uint64_t limit_ns, uint32_t row0, uint32_t col0,
                                             int pieces, uint32_t t_dst, uint8_t *park, int lane, bool vec = true)
{
    if (sig) {
        bool got = true;
        if (lane == 0) got = signal_wait(sig, want, abort_flag, limit_ns);
        got = __shfl_sync(0xFFFFFFFFu, got, 0);
        if (!got) return false;
        __threadfence();
    }
    const uint32_t j = (uint32_t)lane & 7u;
#pragma unroll 1
    for (int i = 0; i < pieces; ++i) {
        const uint32_t col = col0 + (uint32_t)(32 * i) + 4 * j;
        uint32_t v[32];
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint4 x[4];
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const uint32_t grow = row0 + (uint32_t)(16 * half + 4 * it) + ((uint32_t)lane >> 3);
                x[it] = make_uint4(0u, 0u, 0u, 0u);
                if (grow < M && col < N) {
                    const float *src = C + (size_t)grow * N + col;
                    if (vec) {
                        x[it] = __ldcg(reinterpret_cast<const uint4 *>(src));
                    } else {
                        x[it].x = __float_as_uint(__ldcg(src));
                        if (col + 1 < N) x[it].y = __float_as_uint(__ldcg(src + 1));
                        if (col + 2 < N) x[it].z = __float_as_uint(__ldcg(src + 2));
                        if (col + 3 < N) x[it].w = __float_as_uint(__ldcg(src + 3));
                    }
                }
            }
            __syncwarp();                               // the rows parked before have been picked up
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                const uint32_t r = (uint32_t)(4 * it) + ((uint32_t)lane >> 3);
                *reinterpret_cast<uint4 *>(park + r * 128 + ((j ^ (r & 7u)) << 4)) = x[it];
            }
            __syncwarp();
            if ((lane >> 4) == half) {
                const uint8_t *srow = park + (lane & 15) * 128;
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {
                    const uint4 y = *reinterpret_cast<const uint4 *>(srow + ((jj ^ (lane & 7)) << 4));
                    v[4 * jj] = y.x; v[4 * jj + 1] = y.y; v[4 * jj + 2] = y.z; v[4 * jj + 3] = y.w;
                }
            }
        }
        tmem_st_32x32(t_dst + (uint32_t)(i * 32), v);
    }
    __syncwarp();
    tmem_wait_st();
    return true;
}

// Slice of the site table that one warp examines when the CTA builds its list.
struct SiteSlice { int beg, end; };

__device__ __forceinline__ SiteSlice site_slice(int n, int warp)
{
    constexpr int WARPS = NUM_THREADS / 32;
    const int per = ((n + WARPS - 1) / WARPS + 31) / 32 * 32;       // whole 32-entry rounds
    SiteSlice sl;
    sl.beg = min(n, warp * per);
    sl.end = min(n, sl.beg + per);
    return sl;
}

// All threads: ordered list of the valid sites that touch a tile of this CTA (pair). CTA 0 also
// reports invalid entries (skipped) and the applied count. Each warp compacts a contiguous slice
// of the table with ballots, so the list keeps table order. `first` is the entry this thread
// examines in its slice's first round, loaded by the caller ahead of time.
// A table of one entry -- the single fault of a trial (Section IV-A), the usual case -- is handled by warp
// SINGLE_SITE_WARP alone (every lane holds the entry in `first`), with no compaction and no CTA-wide barrier, next
// to the other warps' set-up; it also waits for CTA 0's cleared log where this CTA will write to it.
template <int TM, int BN>
__device__ __noinline__ void build_site_list_many(const GemmParams &p, Control *ctl, uint32_t gid, uint32_t groups, mpgemmfi_site first);

template <int TM, int BN>
__device__ void build_site_list(const GemmParams &p, Control *ctl, uint32_t gid, uint32_t groups,
                                const mpgemmfi_site &first, uint64_t wait_ns)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = p.n_faults;
    if (n == 0) {
        if (tid == 0) { ctl->site_count = 0; ctl->class_end[0] = 0; ctl->class_end[1] = 0; }
        return;
    }
    if (n == 1) {
        if (warp != SINGLE_SITE_WARP) return;
        const bool ok = site_valid(first, p.dtype, p.M, p.N, p.K);
        const bool mine = ok && site_touches_group_warp<TM, BN>(first, p, gid, groups, lane);
        if (lane == 0) {
            ctl->site_count = mine ? 1u : 0u;
            ctl->class_end[0] = (mine && site_class(first.kind) == 0) ? 1u : 0u;
            ctl->class_end[1] = (mine && site_class(first.kind) <= 1) ? 1u : 0u;
            if (mine) { ctl->site_cache[0] = first; ctl->site_idx[0] = 0; }
            if (blockIdx.x == 0) {
                if (!ok) write_log(p, 0, 0u, 0u, 0u, 2u);
                if (p.flags) {
                    if (ok) atomicAdd(&p.flags[3], 1u);
                    else { atomicAdd(&p.flags[4], 1u); atomicOr(&p.flags[0], MPGEMMFI_STATUS_SITE_SKIPPED); }
                }
            } else if (mine && p.flags) {
                signal_wait(p.ready, p.epoch, &ctl->abort_flag, wait_ns);
            }
        }
        return;
    }
    build_site_list_many<TM, BN>(p, ctl, gid, groups, first);
}

template <int TM, int BN>
__device__ __noinline__ void build_site_list_many(const GemmParams &p, Control *ctl, uint32_t gid, uint32_t groups, mpgemmfi_site first)
{
    constexpr int WARPS = NUM_THREADS / 32;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = p.n_faults;
    const SiteSlice sl = site_slice(n, warp);
    uint32_t cnt[3] = {0, 0, 0}, n_valid = 0, n_bad = 0, first_vote = 0;
    for (int base = sl.beg; base < sl.end; base += 32) {
        const int i = base + lane;
        bool ok = false, mine = false;
        int cls = 2;
        if (i < sl.end) {
            const mpgemmfi_site s = base == sl.beg ? first : table_site(p, i);
            ok = site_valid(s, p.dtype, p.M, p.N, p.K);
            mine = ok && site_touches_group<TM, BN>(s, p, gid, groups);
            cls = site_class(s.kind);
            if (!ok && blockIdx.x == 0) write_log(p, i, 0u, 0u, 0u, 2u);
            n_valid += ok ? 1u : 0u;
            n_bad += ok ? 0u : 1u;
        }
        const uint32_t vote = __ballot_sync(0xFFFFFFFFu, mine);
        const uint32_t v0 = __ballot_sync(0xFFFFFFFFu, mine && cls == 0), v1 = __ballot_sync(0xFFFFFFFFu, mine && cls == 1);
        if (base == sl.beg) first_vote = vote;
        cnt[0] += __popc(v0);
        cnt[1] += __popc(v1);
        cnt[2] += __popc(vote) - __popc(v0) - __popc(v1);
    }
    if (blockIdx.x == 0 && p.flags) {
        n_valid = __reduce_add_sync(0xFFFFFFFFu, n_valid);
        n_bad = __reduce_add_sync(0xFFFFFFFFu, n_bad);
        if (lane == 0 && n_valid) atomicAdd(&p.flags[3], n_valid);
        if (lane == 0 && n_bad) { atomicAdd(&p.flags[4], n_bad); atomicOr(&p.flags[0], MPGEMMFI_STATUS_SITE_SKIPPED); }
    }
    if (lane == 0) { ctl->scan[0][warp] = cnt[0]; ctl->scan[1][warp] = cnt[1]; ctl->scan[2][warp] = cnt[2]; }
    __syncthreads();
    // where this warp's entries of each class go: after the classes before it and, inside the class, after the
    // entries of the warps before it (their slices of the table come first)
    uint32_t off[3], total[3];
#pragma unroll
    for (int c = 0; c < 3; ++c) {
        off[c] = 0; total[c] = 0;
        for (int w = 0; w < WARPS; ++w) {
            const uint32_t x = ctl->scan[c][w];
            if (w < warp) off[c] += x;
            total[c] += x;
        }
    }
    off[1] += total[0];
    off[2] += total[0] + total[1];
    if (tid == 0) {
        ctl->class_end[0] = total[0];
        ctl->class_end[1] = total[0] + total[1];
        ctl->site_count = total[0] + total[1] + total[2];
    }
    for (int base = sl.beg; base < sl.end; base += 32) {
        const int i = base + lane;
        bool mine = false;
        mpgemmfi_site s = first;
        if (base != sl.beg) {
            if (i < sl.end) {
                s = table_site(p, i);
                mine = site_valid(s, p.dtype, p.M, p.N, p.K) && site_touches_group<TM, BN>(s, p, gid, groups);
            }
        } else {
            mine = (first_vote >> lane) & 1u;
        }
        const int cls = site_class(s.kind);
        const uint32_t lower = (1u << lane) - 1u;
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            const uint32_t vc = __ballot_sync(0xFFFFFFFFu, mine && cls == c);
            if (mine && cls == c) {
                const uint32_t pos = off[c] + __popc(vc & lower);
                if (pos < (uint32_t)SITE_CACHE) ctl->site_cache[pos] = s;
                ctl->site_idx[pos] = (uint16_t)i;
            }
            off[c] += __popc(vc);
        }
    }
}

// two FP32 words -> one word holding their roundings (to nearest, ties to even) to the 16-bit output format,
// the first in the low half
__device__ __forceinline__ uint32_t pack_out16(int out_fmt, uint32_t lo_bits, uint32_t hi_bits)
{
    if (out_fmt == MPGEMMFI_OUT_FP16) {
        const __half2 h = __floats2half2_rn(bits_f32(lo_bits), bits_f32(hi_bits));
        return *reinterpret_cast<const uint32_t *>(&h);
    }
    const __nv_bfloat162 b = __floats2bfloat162_rn(bits_f32(lo_bits), bits_f32(hi_bits));
    return *reinterpret_cast<const uint32_t *>(&b);
}

// kPair = false: grid of single CTAs, tiles 128 x BN.
// kPair = true : grid of CTA pairs (cluster dimension 2), tiles 256 x BN, BN = 256.
template <int BN, bool kTF32, bool kPair>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
            const __grid_constant__ CUtensorMap tm_c, const __grid_constant__ GemmParams p)
{
    using C = Cfg<BN, kPair>;
    constexpr int KT = kTF32 ? 32 : 64;      // elements per 128-byte row
    constexpr int STAGES = C::STAGES;
    constexpr int TM = kPair ? 2 * BM : BM;  // rows of one tile
    constexpr uint32_t EPI_ARRIVALS = kPair ? 2 * EPI_WARPS : EPI_WARPS;   // one arrival per epilogue warp

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t *stage_out = smem + STAGES * C::STAGE_BYTES;     // output staging of the epilogue warps
    Control *ctl = reinterpret_cast<Control *>(stage_out + OUT_STAGING_BYTES);
    volatile uint32_t *abort_flag = &ctl->abort_flag;
    const uint64_t wait_ns = p.wait_limit_ns;       // how long any one wait below may last before the CTA gives up

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = kPair ? cluster_cta_rank() : 0u;          // 0 = leader of the pair
    const uint32_t gid = kPair ? blockIdx.x >> 1 : blockIdx.x;      // tile walker id
    const uint32_t groups = kPair ? gridDim.x >> 1 : gridDim.x;
    const bool leader = rank == 0;

    // this thread's first entry of the site table: requested now, needed only after the set-up below
    mpgemmfi_site first_site = {};
    if (p.n_faults == 1) {
        if (warp == SINGLE_SITE_WARP) first_site = table_site(p, 0);
    } else if (p.n_faults > 0) {
        const SiteSlice sl = site_slice(p.n_faults, warp);
        if (sl.beg + lane < sl.end) first_site = table_site(p, sl.beg + lane);
    }
    // (set by the thread that may be the first to poll it, see build_site_list; everybody else meets it after a barrier)
    if (threadIdx.x == SINGLE_SITE_WARP * 32) ctl->abort_flag = 0;

    if (blockIdx.x == 0 && p.flags) {
        // header and site log start at zero: cleared here rather than by a memset in front of every launch
        // (2.5 us each); the other CTAs learn through *p.ready that it has been done
        for (uint32_t i = threadIdx.x; i < (uint32_t)(MPGEMMFI_HEADER_WORDS + 4 * p.n_faults); i += NUM_THREADS) p.flags[i] = 0u;
        __syncthreads();
        if (threadIdx.x == 0) { __threadfence(); signal_store_release(p.ready, p.epoch); }
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            // pair mode, leader CTA: one arrival per CTA of the pair (each announces its own bytes)
            mbar_init(smem_u32(&ctl->full[s]), (kPair && leader) ? 2 : 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->acc_full[s]), 1); mbar_init(smem_u32(&ctl->acc_empty[s]), EPI_ARRIVALS); }
        mbar_init(smem_u32(&ctl->pause_full), 1);
        mbar_init(smem_u32(&ctl->pause_done), EPI_ARRIVALS);
        for (int s = 0; s < 2; ++s) mbar_init(smem_u32(&ctl->acc_loaded[s]), EPI_ARRIVALS);
        mbar_fence_init();
        tma_prefetch_desc(&tm_a);
        tma_prefetch_desc(&tm_b);
        if (p.c_vec_ok) tma_prefetch_desc(&tm_c);
    }
    if (warp == 2) {
        if constexpr (kPair) { tmem_alloc_pair(smem_u32(&ctl->tmem_base), C::TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&ctl->tmem_base), C::TMEM_COLS); tmem_relinquish(); }
    }
    build_site_list<TM, BN>(p, ctl, gid, groups, first_site, wait_ns);
    // a CTA with sites writes log entries as it goes: not before CTA 0 has cleared the log
    // (a one-entry table: waited for inside build_site_list)
    if (threadIdx.x == 0 && blockIdx.x != 0 && p.flags && p.n_faults > 1 && ctl->site_count != 0)
        signal_wait(p.ready, p.epoch, abort_flag, wait_ns);
    tc_fence_before_sync();
    if constexpr (kPair) cluster_sync_all(); else __syncthreads();
    tc_fence_after_sync();

    const uint32_t tmem_base = ctl->tmem_base;
    const bool has_sites = ctl->site_count != 0;
    TileCtx tc;
    tc.p = &p; tc.ctl = ctl; tc.bn = BN; tc.tile_rows = TM; tc.b_rows = C::B_ROWS;
    auto set_tile = [&](uint32_t t) {
        uint32_t tm, tn;
        tile_coords(p, t, tm, tn);
        tc.tile_m0 = tm * TM;
        tc.m0 = tc.tile_m0 + rank * BM;
        tc.n0 = tn * BN;
        tc.b0 = tc.n0 + rank * C::B_ROWS;
    };
    // barriers of the leader CTA that this CTA's warps arrive on
    const uint32_t lead_acc_empty0 = kPair ? map_to_cta(smem_u32(&ctl->acc_empty[0]), 0) : smem_u32(&ctl->acc_empty[0]);
    const uint32_t lead_pause_done = kPair ? map_to_cta(smem_u32(&ctl->pause_done), 0) : smem_u32(&ctl->pause_done);
    const uint32_t lead_acc_loaded0 = kPair ? map_to_cta(smem_u32(&ctl->acc_loaded[0]), 0) : smem_u32(&ctl->acc_loaded[0]);
    Segment sg;

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        // Pair mode: both CTAs count their bytes on the LEADER's full barrier, so the leader's MMA
        // warp waits on one barrier per stage. Exception: a stage in which the non-leader CTA has
        // an operand site is loaded against that CTA's own barrier; its warp 1 flips the element
        // and then delivers the CTA's arrival to the leader.
        uint32_t stage = 0, phase = 0, armed = 0, armed_parity = 0;
        const uint32_t lead_full0 = kPair ? map_to_cta(smem_u32(&ctl->full[0]), 0) : 0u;
        bool ok = true;
        for (uint32_t si = 0; ok && get_segment(p, gid, groups, si, sg); ++si) {
            set_tile(sg.tile);
            uint32_t next_op = NONE;
            if (kPair && !leader && has_sites) next_op = scan_next_operand(tc, sg.kt0, lane);
            for (uint32_t kt = sg.kt0; kt < sg.kt1; ++kt) {
                const bool own_barrier = !kPair || leader || kt == next_op;
                if (kPair && kt == next_op) next_op = scan_next_operand(tc, kt + 1, lane);
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&ctl->empty[stage]), phase ^ 1u, abort_flag, wait_ns);
                    if (ok) {
                        uint8_t *sa = smem + stage * C::STAGE_BYTES;
                        if (own_barrier) {
                            const uint32_t bar = smem_u32(&ctl->full[stage]);
                            mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                            tma_load_2d(smem_u32(sa), &tm_a, bar, (int)(kt * KT), (int)tc.m0);
                            tma_load_2d(smem_u32(sa + C::A_BYTES), &tm_b, bar, (int)(kt * KT), (int)tc.b0);
                            armed |= 1u << stage;
                            armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
                        } else {
                            const uint32_t bar = lead_full0 + stage * (uint32_t)sizeof(uint64_t);
                            mbar_arrive_expect_tx_cluster(bar, C::STAGE_BYTES);
                            tma_load_2d_pair(smem_u32(sa), &tm_a, bar, (int)(kt * KT), (int)tc.m0);
                            tma_load_2d_pair(smem_u32(sa + C::A_BYTES), &tm_b, bar, (int)(kt * KT), (int)tc.b0);
                        }
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                if (!ok) break;
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
        // wait (bounded) until every copy counted on this CTA's barriers has landed (the leader's
        // barriers also count the other CTA's copies)
        if (lane == 0 && (!kPair || leader)) {
            uint32_t never = 0;
            for (int s = 0; s < STAGES; ++s)
                if (armed & (1u << s))
                    mbar_wait(smem_u32(&ctl->full[s]), (armed_parity >> s) & 1u, &never, 1000000000ull);
        }
    } else if (warp == 1 && !leader) {
        // ------------------------------------------------------------ pair mode, non-leader CTA: no MMAs to
        // issue; only the stages that carry one of this CTA's operand sites need attention
        if (has_sites) {
            uint32_t steps_before = 0, own_phase = 0;     // own_phase: bit s = parity of this CTA's full[s]
            bool ok = true;
            const uint32_t lead_full0 = map_to_cta(smem_u32(&ctl->full[0]), 0);
            for (uint32_t si = 0; ok && get_segment(p, gid, groups, si, sg); steps_before += sg.kt1 - sg.kt0, ++si) {
                set_tile(sg.tile);
                uint32_t kt = scan_next_operand(tc, sg.kt0, lane);
                while (kt < sg.kt1) {          // NONE is larger than any k-tile
                    const uint32_t g = steps_before + (kt - sg.kt0), stage = g % STAGES;
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->full[stage]), (own_phase >> stage) & 1u, abort_flag, wait_ns));
                    if (!ok) break;
                    own_phase ^= 1u << stage;
                    {
                        uint8_t *sa = smem + stage * C::STAGE_BYTES;
                        apply_operand_sites(tc, kt, sa, sa + C::A_BYTES, lane);
                    }
                    if (lane == 0) {
                        fence_proxy_async_smem();
                        mbar_arrive_cluster(lead_full0 + stage * (uint32_t)sizeof(uint64_t));
                    }
                    __syncwarp();
                    kt = scan_next_operand(tc, kt + 1, lane);
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        const uint32_t idesc = umma_instr_desc((uint32_t)p.dtype, TM, BN);
        uint32_t stage = 0, phase = 0, pause_phase = 0, loaded_phase = 0;
        bool ok = true;
        for (uint32_t lt = 0; ok && get_segment(p, gid, groups, lt, sg); ++lt) {
            const uint32_t as = lt & 1u, ap = (lt >> 1) & 1u;
            set_tile(sg.tile);
            uint32_t next_op = NONE, next_b = NONE;
            if (has_sites) { next_op = scan_next_operand(tc, sg.kt0, lane); next_b = scan_next_boundary(tc, sg.kt0 + 1, lane); }
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->acc_empty[as]), ap ^ 1u, abort_flag, wait_ns));
            if (!ok) break;
            const bool preloaded = starts_from_memory(p, sg);
            if (preloaded) {
                // continued tile or addend: the epilogue warps put the starting accumulators into TMEM first
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->acc_loaded[as]), (loaded_phase >> as) & 1u, abort_flag, wait_ns));
                if (!ok) break;
                loaded_phase ^= 1u << as;
            }
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + as * BN;
            const uint32_t fresh_kt = preloaded ? NONE : sg.kt0;    // the k-tile whose first MMA overwrites the accumulator
            uint32_t kt = sg.kt0;
            while (kt < sg.kt1) {
              // k-tiles up to the next one with a site (an operand site in it, or an accumulator / term site
              // at the boundary behind it) -- usually all of them: one thread runs the loop, with no
              // warp-wide step in it, so that issuing a k-tile's MMAs takes less time than the tensor core
              // needs to run them
              const uint32_t stop = min(sg.kt1, min(next_op, next_b - 1u));
              if (kt < stop) {
                if (lane == 0) {
                    const uint32_t full0 = smem_u32(&ctl->full[0]), empty0 = smem_u32(&ctl->empty[0]);
                    const uint64_t desc0 = umma_smem_desc_sw128(smem_u32(smem));
                    uint32_t accumulate = kt == fresh_kt ? 0u : 1u;
                    for (; kt < stop; ++kt) {
                        if (!mbar_wait(full0 + stage * 8u, phase, abort_flag, wait_ns)) { ok = false; break; }
                        tc_fence_after_sync();
                        // the address field counts 16-byte units: stage s starts s * STAGE_BYTES / 16 further on
                        const uint64_t a_desc = desc0 + (uint64_t)(stage * (uint32_t)(C::STAGE_BYTES >> 4));
                        const uint64_t b_desc = a_desc + (uint64_t)(C::A_BYTES >> 4);
#pragma unroll
                        for (uint32_t k = 0; k < 4; ++k) {
                            if constexpr (kPair) umma_ss_pair<kTF32>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                            else umma_ss<kTF32>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                            accumulate = 1u;
                        }
                        if constexpr (kPair) umma_commit_pair(empty0 + stage * 8u, 3);
                        else umma_commit(empty0 + stage * 8u);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                stage = __shfl_sync(0xFFFFFFFFu, stage, 0);
                phase = __shfl_sync(0xFFFFFFFFu, phase, 0);
                if (!ok) break;
                kt = stop;
                continue;
              }
              // one k-tile with a site, by the whole warp
              {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->full[stage]), phase, abort_flag, wait_ns));
                if (!ok) break;
                tc_fence_after_sync();
                uint8_t *sa = smem + stage * C::STAGE_BYTES;
                if (kt == next_op) {
                    apply_operand_sites(tc, kt, sa, sa + C::A_BYTES, lane);
                    if (lane == 0) fence_proxy_async_smem();
                    __syncwarp();
                }
                if (lane == 0) {
                    const uint64_t a_desc = umma_smem_desc_sw128(smem_u32(sa));
                    const uint64_t b_desc = umma_smem_desc_sw128(smem_u32(sa + C::A_BYTES));
#pragma unroll
                    for (uint32_t k = 0; k < 4; ++k) {   // 4 x 32 bytes along K inside the swizzle row
                        const uint32_t accumulate = (kt == fresh_kt && k == 0) ? 0u : 1u;
                        if constexpr (kPair) umma_ss_pair<kTF32>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                        else umma_ss<kTF32>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                    }
                    if constexpr (kPair) umma_commit_pair(smem_u32(&ctl->empty[stage]), 3);
                    else umma_commit(smem_u32(&ctl->empty[stage]));
                }
                __syncwarp();
                if (kt == next_op) next_op = scan_next_operand(tc, kt + 1, lane);     // (after the MMAs are on their way)
                if (kt + 1 == next_b) {
                    // an accumulator / term site takes effect here: let the epilogue warps edit TMEM
                    if (lane == 0) {
                        if constexpr (kPair) umma_commit_pair(smem_u32(&ctl->pause_full), 3);
                        else umma_commit(smem_u32(&ctl->pause_full));
                    }
                    __syncwarp();
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->pause_done), pause_phase, abort_flag, wait_ns));
                    if (!ok) break;
                    pause_phase ^= 1u;
                    tc_fence_after_sync();
                    next_b = scan_next_boundary(tc, kt + 2, lane);
                }
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                ++kt;
              }
            }
            if (!ok) break;
            if (lane == 0) {
                if constexpr (kPair) umma_commit_pair(smem_u32(&ctl->acc_full[as]), 3);
                else umma_commit(smem_u32(&ctl->acc_full[as]));
            }
            __syncwarp();
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ epilogue (own 128 rows)
        const int q = warp & 3;               // TMEM lane quarter this warp may access
        const int h = (warp - 4) >> 2;        // column half of the tile this warp handles
        const int tech = p.detect_mode & MPGEMMFI_DETECT_TECHNIQUE_MASK;
        const bool want_bound = tech == MPGEMMFI_DETECT_BOUNDCHECK;
        const bool want_range = (p.detect_mode & MPGEMMFI_OUTPUT_RANGE) && p.exp_a != nullptr &&
                                (tech == MPGEMMFI_DETECT_RANGE_MAX || tech == MPGEMMFI_DETECT_RANGE_FLIP);
        const bool range_flip = tech == MPGEMMFI_DETECT_RANGE_FLIP;
        const bool want_corr = (want_bound || want_range) && (p.detect_mode & MPGEMMFI_CORRECT);
        // The per-element work of a tile is compiled once per check mode (EPI_*), so that the 32-element
        // loops carry no mode tests: left to itself the compiler does not always pull them out of the
        // tile loop (when it did not, a launch ran a quarter more instructions).
        const int epi_mode = want_range ? EPI_RANGE : (want_bound ? (want_corr ? EPI_BOUND_CORRECT : EPI_BOUND) : EPI_PLAIN);
        uint32_t pause_phase = 0, n_det = 0;
        uint32_t *bitmap = p.flags ? p.flags + MPGEMMFI_HEADER_WORDS + 4 * (size_t)p.n_faults : nullptr;
        uint8_t *my_out = stage_out + (warp - 4) * OUT_BUF_BYTES;
        // where this thread parks 16-byte chunk j of its row for a TMA store: park_addr ^ (j << 4) (128-byte swizzle:
        // chunk j of row r sits at chunk position j ^ (r & 7))
        const uint32_t park_addr = smem_u32(my_out) + ((uint32_t)lane & 15u) * 128u + (((uint32_t)lane & 7u) << 4);
        // the same for a 16-bit output: rows of 64 bytes, 64-byte swizzle (chunk c of row r at position c ^ ((r >> 1) & 3))
        const uint32_t park16_addr = smem_u32(my_out) + (uint32_t)lane * 64u + ((((uint32_t)lane >> 1) & 3u) << 4);
        constexpr int MY_PIECES = BN / 64;          // 32-column pieces per warp (half the tile's columns)
        const int first = h * MY_PIECES;
        // hand-over words of this warp for left-over tile j: signals[j * 16 + my_signal]
        const uint32_t my_signal = rank * EPI_WARPS + (uint32_t)(warp - 4);
        const uint32_t first_left = groups * (uint32_t)p.full_rounds;
        bool ok = true;
        // This warp's share of what segment s starts from, into accumulator buffer `buf`: the sums the walker
        // of the previous part left in C (after that walker's hand-over), or the addend.
        auto preload = [&](const Segment &s, uint32_t buf) -> bool {
            uint32_t tm, tn;
            tile_coords(p, s.tile, tm, tn);
            if (lane == 0) bulk_wait_read_all();       // the staging rows are free again
            __syncwarp();
            const uint32_t *sig = s.load ? p.signals + (size_t)(s.tile - first_left) * 16 + my_signal : nullptr;
            const uint32_t t_dst = tmem_base + buf * BN + ((uint32_t)(q * 32) << 16) + (uint32_t)(first * 32);
            // (p.tag_skew is zero outside the tests, see GemmParams)
            if (!load_partial(s.load ? p.C : p.addend, (uint32_t)p.M, (uint32_t)p.N, sig, ((p.epoch << 3) | s.part) ^ p.tag_skew,
                              abort_flag, wait_ns, tm * TM + rank * BM + (uint32_t)(q * 32), tn * BN + (uint32_t)(first * 32), MY_PIECES,
                              t_dst, my_out, lane, s.load || p.addend_vec_ok != 0))
                return false;
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                if constexpr (kPair) mbar_arrive_cluster(lead_acc_loaded0 + buf * (uint32_t)sizeof(uint64_t));
                else mbar_arrive(lead_acc_loaded0 + buf * (uint32_t)sizeof(uint64_t));
            }
            return true;
        };
        if (p.addend != nullptr && get_segment(p, gid, groups, 0, sg) && starts_from_memory(p, sg)) ok = preload(sg, 0u);
        for (uint32_t lt = 0; ok && get_segment(p, gid, groups, lt, sg); ++lt) {
            const uint32_t as = lt & 1u, ap = (lt >> 1) & 1u;
            if (p.split_parts > 1 || p.addend != nullptr) {
                // the other TMEM buffer is free (this warp has read its share of the segment before this
                // one): if the next segment starts from memory, fetch its accumulators while this one runs
                Segment nx;
                if (get_segment(p, gid, groups, lt + 1, nx) && starts_from_memory(p, nx)) {
                    ok = preload(nx, (lt + 1) & 1u);
                    if (!ok) break;
                }
            }
            set_tile(sg.tile);
            // the walker's last piece of work: when its accumulators are complete the operand ring is free (see
            // store_piece_tail)
            bool last_seg;
            {
                Segment nx;
                last_seg = !get_segment(p, gid, groups, lt + 1, nx);
            }
            const uint32_t tmem_acc = tmem_base + as * BN;
            bool tile_has_out = false;
            if (has_sites) {
                uint32_t b = scan_next_boundary(tc, sg.kt0 + 1, lane);
                while (b <= sg.kt1) {          // boundaries of this segment's k-tiles (NONE is larger than any)
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->pause_full), pause_phase, abort_flag, wait_ns));
                    if (!ok) break;
                    pause_phase ^= 1u;
                    tc_fence_after_sync();
                    apply_boundary_sites(tc, b, tmem_acc, q, h, lane);
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        if constexpr (kPair) mbar_arrive_cluster(lead_pause_done);
                        else mbar_arrive(lead_pause_done);
                    }
                    b = scan_next_boundary(tc, b + 1, lane);
                }
                if (!ok) break;
                tile_has_out = !sg.save && scan_has_out(tc, lane);
            }
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&ctl->acc_full[as]), ap, abort_flag, wait_ns));
            if (!ok) break;
            tc_fence_after_sync();

            const uint32_t row = tc.m0 + (uint32_t)(q * 32 + lane);
            const uint32_t row0 = tc.m0 + (uint32_t)(q * 32);
            const bool row_ok = row < (uint32_t)p.M;
            float *crow = p.C + (size_t)row * p.N;
            const uint32_t t_first = tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)(first * 32);

            // stores of one 32-column piece (this thread's row, columns c0..c0+31) to C
            auto store_piece = [&](uint32_t (&v)[32], uint32_t c0) {
                if (p.c_vec_ok) {
                    // Transpose through shared memory so that every store instruction writes whole
                    // 128-byte rows, 16 rows at a time: threads of one half-warp park their rows
                    // (16-byte piece j of row r in slot j ^ (r & 7), conflict-free), then lane l stores
                    // piece l % 8 of rows l / 8 + 4 i.
                    const uint32_t j = (uint32_t)lane & 7u;
                    const uint32_t col = c0 + 4 * j;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        __syncwarp();                           // the previous rows have been read back
                        if ((lane >> 4) == half) {
                            uint8_t *srow = my_out + (lane & 15) * 128;
#pragma unroll
                            for (int jj = 0; jj < 8; ++jj)
                                *reinterpret_cast<uint4 *>(srow + ((jj ^ (lane & 7)) << 4)) =
                                    make_uint4(v[4 * jj], v[4 * jj + 1], v[4 * jj + 2], v[4 * jj + 3]);
                        }
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 4; ++it) {
                            const uint32_t r = (uint32_t)(4 * it) + ((uint32_t)lane >> 3);      // row within the 16
                            const uint4 val = *reinterpret_cast<const uint4 *>(my_out + r * 128 + ((j ^ (r & 7u)) << 4));
                            const uint32_t grow = row0 + (uint32_t)(16 * half) + r;
                            if (grow < (uint32_t)p.M && col < (uint32_t)p.N)
                                *reinterpret_cast<uint4 *>(p.C + (size_t)grow * p.N + col) = val;
                        }
                    }
                } else if (row_ok) {
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj)
                        if (c0 + jj < (uint32_t)p.N) crow[c0 + jj] = bits_f32(v[jj]);
                }
            };
            // The same for a finished tile when C allows 16-byte accesses: the rows are parked in the layout of the
            // 128-byte swizzle and one thread hands them to the TMA engine (16 rows x 128 bytes a store, the two
            // half-warps in turn). The warp does not wait for the store, only -- before it parks the next rows -- for
            // its staging to have been read: the SM's write port (about 32 bytes a cycle) then drains one warp's rows
            // while the other warps check and park theirs, instead of all eight warps checking together and then
            // queueing behind the port together.
            auto store_piece_tma = [&](uint32_t (&v)[32], uint32_t c0) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (lane == 0) bulk_wait_read_all();
                    __syncwarp();
                    if ((lane >> 4) == half) {
#pragma unroll
                        for (int jj = 0; jj < 8; ++jj)
                            st_shared_v4(park_addr ^ (uint32_t)(jj << 4), v[4 * jj], v[4 * jj + 1], v[4 * jj + 2], v[4 * jj + 3]);
                        fence_proxy_async_smem();
                    }
                    __syncwarp();
                    const uint32_t r0 = row0 + (uint32_t)(16 * half);
                    if (lane == 0 && r0 < (uint32_t)p.M && c0 < (uint32_t)p.N) {
                        tma_store_2d(&tm_c, smem_u32(my_out), (int)c0, (int)r0);
                        bulk_commit_group();
                    }
                }
            };
            // The same for the walker's LAST tile. Nothing overlaps that tile's epilogue, so its latency is the launch's
            // tail; and once its accumulators are complete (acc_full: every MMA of this CTA, or pair, has read its
            // operands) the operand ring is free. Every piece gets 4 KB of it to itself: all 32 threads park their rows
            // at once and both 16-row stores leave without any wait for an earlier store to have read the staging.
            auto store_piece_tail = [&](uint32_t (&v)[32], uint32_t c0, int piece) {
                const uint32_t buf = smem_u32(smem) + ((uint32_t)(warp - 4) * (uint32_t)MY_PIECES + (uint32_t)piece) * 4096u;
                const uint32_t mine = buf + (uint32_t)lane * 128u;
#pragma unroll
                for (int jj = 0; jj < 8; ++jj)
                    st_shared_v4(mine + ((uint32_t)(jj ^ (lane & 7)) << 4), v[4 * jj], v[4 * jj + 1], v[4 * jj + 2], v[4 * jj + 3]);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && c0 < (uint32_t)p.N) {
                    if (row0 < (uint32_t)p.M) tma_store_2d(&tm_c, buf, (int)c0, (int)row0);
                    if (row0 + 16 < (uint32_t)p.M) tma_store_2d(&tm_c, buf + 2048u, (int)c0, (int)(row0 + 16));
                    bulk_commit_group();
                }
            };
            // 16-bit output: the checked FP32 values are rounded once (to nearest even) and the whole 32 x 32 piece, now
            // 64 bytes a row, fits the staging: all 32 threads park their rows at once and the piece leaves as ONE store.
            auto store_piece16 = [&](uint32_t (&v)[32], uint32_t c0, int piece) {
                uint32_t h[16];
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) h[jj] = pack_out16(p.out_fmt, v[2 * jj], v[2 * jj + 1]);
                if (p.c_vec_ok) {
                    // the walker's last tile: a buffer of the free operand ring per piece, no wait (see store_piece_tail)
                    const uint32_t buf = last_seg ? smem_u32(smem) + ((uint32_t)(warp - 4) * (uint32_t)MY_PIECES + (uint32_t)piece) * 2048u
                                                  : smem_u32(my_out);
                    if (!last_seg) {
                        if (lane == 0) bulk_wait_read_all();
                        __syncwarp();
                    }
                    const uint32_t mine = buf + (park16_addr - smem_u32(my_out));
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        st_shared_v4(mine ^ (uint32_t)(c << 4), h[4 * c], h[4 * c + 1], h[4 * c + 2], h[4 * c + 3]);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && row0 < (uint32_t)p.M && c0 < (uint32_t)p.N) {
                        tma_store_2d(&tm_c, buf, (int)c0, (int)row0);
                        bulk_commit_group();
                    }
                } else if (row_ok) {
                    unsigned short *drow = reinterpret_cast<unsigned short *>(p.C) + (size_t)row * p.N;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj)
                        if (c0 + jj < (uint32_t)p.N) drow[c0 + jj] = (unsigned short)(h[jj >> 1] >> (16 * (jj & 1)));
                }
            };
            // accumulator columns of this warp fully read: one arrival towards handing the TMEM
            // buffer back to the MMA warp
            auto release_acc = [&]() {
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (kPair) mbar_arrive_cluster(lead_acc_empty0 + as * (uint32_t)sizeof(uint64_t));
                    else mbar_arrive(lead_acc_empty0 + as * (uint32_t)sizeof(uint64_t));
                }
            };

            if (sg.save) {
                // unfinished tile: the raw accumulators go to the tile's place in C (no output site, no check),
                // then the walker of the next part is told that this warp's share is there
                if (lane == 0) bulk_wait_read_all();
                __syncwarp();
#pragma unroll 1
                for (int i = 0; i < MY_PIECES; ++i) {
                    uint32_t raw[32];
                    tmem_ld_32x32(t_first + (uint32_t)(i * 32), raw);
                    tmem_wait_ld();
                    store_piece(raw, tc.n0 + (uint32_t)((first + i) * 32));
                }
                release_acc();
                __threadfence();
                __syncwarp();
                if (lane == 0)
                    signal_store_release(p.signals + (size_t)(sg.tile - first_left) * 16 + my_signal, (p.epoch << 3) | (sg.part + 1u));
                continue;
            }

            // The finished tile under check mode kMode (a compile-time constant inside).
            auto finish_tile = [&](auto mode_tag) {
                constexpr int kMode = decltype(mode_tag)::value;
                constexpr bool do_bound = kMode == EPI_BOUND || kMode == EPI_BOUND_CORRECT;
                constexpr bool do_range = kMode == EPI_RANGE;
                const bool do_corr = kMode == EPI_BOUND_CORRECT || (kMode == EPI_RANGE && want_corr);
                const uint32_t row_e = (do_range && row_ok) ? __ldg(p.exp_a + row) : 0u;

                // One 32-column piece of this thread's row: output sites, check, flags, store.
                auto finish_piece = [&](uint32_t (&v)[32], int i) -> uint32_t {
                    const uint32_t c0 = tc.n0 + (uint32_t)((first + i) * 32);
                    // output-level range check: this lane fetches the exponent maximum of column c0 + lane early
                    uint32_t col_e = 0;
                    if (do_range && c0 + (uint32_t)lane < (uint32_t)p.N) col_e = __ldg(p.exp_b + c0 + lane);
                    if (tile_has_out && row_ok) apply_out_sites(tc, row, c0, v, 0);
                    uint32_t fw = 0;
                    if constexpr (do_range) {
                        const int row_part = (int)row_e - 126 + p.log2_k;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int bound = min(255, max(0, row_part + (int)__shfl_sync(0xFFFFFFFFu, col_e, j)));
                            const bool det = (int)((v[j] >> 23) & 0xFFu) > bound;
                            if (det) {
                                fw |= 1u << j;
                                if (do_corr) v[j] = range_flip ? rangecheck_flip(v[j], bound) : rangecheck_max(v[j], bound);
                            }
                        }
                        if (c0 + 32 > (uint32_t)p.N) fw &= c0 < (uint32_t)p.N ? (1u << ((uint32_t)p.N - c0)) - 1u : 0u;
                    }
                    if constexpr (do_bound) {
                        // A flagged element has exponent bit 7 (word bit 30) set. The OR of the 32 words costs a
                        // third of the per-element test and settles the usual case (every |value| < 2) at once.
                        uint32_t o8[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) o8[j] = (v[4 * j] | v[4 * j + 1]) | (v[4 * j + 2] | v[4 * j + 3]);
                        const uint32_t any = ((o8[0] | o8[1]) | (o8[2] | o8[3])) | ((o8[4] | o8[5]) | (o8[6] | o8[7]));
                        if (any & 0x40000000u) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                // exponent field >= 0x90 <=> not (|value| < 131072); NaN compares false, so it is caught
                                const bool det = !(fabsf(bits_f32(v[j])) < 131072.0f);
                                if (det) fw |= 1u << j;
                                if (kMode == EPI_BOUND_CORRECT && det) v[j] = boundcheck_clear(v[j]);
                            }
                        }
                        // columns past N are not part of C (their zero-filled Bt rows still give NaN against an
                        // Inf or NaN in A): their flag bits stay 0
                        if (c0 + 32 > (uint32_t)p.N) fw &= c0 < (uint32_t)p.N ? (1u << ((uint32_t)p.N - c0)) - 1u : 0u;
                    }
                    if (tile_has_out && row_ok) apply_out_sites(tc, row, c0, v, 1);
                    if (p.out_fmt != MPGEMMFI_OUT_FP32) store_piece16(v, c0, i);
                    else if (p.c_vec_ok && last_seg) store_piece_tail(v, c0, i);
                    else if (p.c_vec_ok) store_piece_tma(v, c0);
                    else store_piece(v, c0);
                    return fw;
                };

                // Software pipeline: the TMEM read of the next piece is in flight while this one is finished. Two
                // pieces per trip of a loop that is NOT unrolled: the epilogue's code stays a quarter of what four
                // inlined copies take, which is what the instruction cache can hold next to the other warps' loops.
                uint32_t va[32], vb[32];
                tmem_ld_32x32(t_first, va);
                uint32_t *frow = nullptr;
                const uint32_t w0 = tc.n0 / 32 + (uint32_t)first;
                if (bitmap && row_ok) frow = bitmap + (size_t)row * p.wpr + w0;
#pragma unroll 1
                for (int i = 0; i < MY_PIECES; i += 2) {
                    tmem_wait_ld();
                    if (i + 1 < MY_PIECES) tmem_ld_32x32(t_first + (uint32_t)((i + 1) * 32), vb);
                    else release_acc();
                    const uint32_t fa = finish_piece(va, i);
                    uint32_t fb = 0;
                    if (i + 1 < MY_PIECES) {
                        tmem_wait_ld();
                        if (i + 2 < MY_PIECES) tmem_ld_32x32(t_first + (uint32_t)((i + 2) * 32), va);
                        else release_acc();
                        fb = finish_piece(vb, i + 1);
                    }
                    if (frow) {
                        if (MY_PIECES > 1 && (p.wpr & 1) == 0) {          // this thread's two words are 8-byte aligned
                            if (w0 + i < (uint32_t)p.wpr) *reinterpret_cast<uint2 *>(frow + i) = make_uint2(fa, fb);
                        } else {
                            if (w0 + i < (uint32_t)p.wpr) frow[i] = fa;
                            if (i + 1 < MY_PIECES && w0 + i + 1 < (uint32_t)p.wpr) frow[i + 1] = fb;
                        }
                        n_det += __popc(fa) + __popc(fb);
                    }
                }
            };
            switch (epi_mode) {
            case EPI_PLAIN: finish_tile(std::integral_constant<int, EPI_PLAIN>{}); break;
            case EPI_BOUND: finish_tile(std::integral_constant<int, EPI_BOUND>{}); break;
            case EPI_BOUND_CORRECT: finish_tile(std::integral_constant<int, EPI_BOUND_CORRECT>{}); break;
            default: finish_tile(std::integral_constant<int, EPI_RANGE>{}); break;
            }
        }
        if (lane == 0) bulk_wait_read_all();       // shared memory stays until the last store has read it
        n_det = __reduce_add_sync(0xFFFFFFFFu, n_det);
        if (lane == 0 && n_det && p.flags && (blockIdx.x == 0 || signal_wait(p.ready, p.epoch, abort_flag, wait_ns))) {
            atomicAdd(&p.flags[1], n_det);
            if (want_corr) atomicAdd(&p.flags[2], n_det);
        }
    }

    tc_fence_before_sync();
    // nobody leaves while the other CTA of a pair may still read this CTA's shared memory,
    // arrive on its barriers or use the shared TMEM allocation
    if constexpr (kPair) cluster_sync_all(); else __syncthreads();
    if (warp == 2) {
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
        else tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
    if (threadIdx.x == 0 && ctl->abort_flag && p.flags) {
        if (blockIdx.x != 0) { volatile uint32_t never = 0; signal_wait(p.ready, p.epoch, &never, 1000000000ull); }
        atomicOr(&p.flags[0], MPGEMMFI_STATUS_WAIT_LIMIT);
    }
    if (threadIdx.x == 0 && blockIdx.x == 0 && p.flags && p.split_parts > 1) p.flags[5] = (uint32_t)p.split_parts;
}

template <int BN, bool kTF32, bool kPair>
cudaError_t launch_one(const CUtensorMap &tm_a, const CUtensorMap &tm_b, const CUtensorMap &tm_c, const GemmParams &p,
                       int grid, cudaStream_t stream)
{
    using C = Cfg<BN, kPair>;
    const size_t smem = (size_t)C::STAGES * C::STAGE_BYTES + OUT_STAGING_BYTES + sizeof(Control) + 1024;
    static_assert(C::STAGES * C::STAGE_BYTES + OUT_STAGING_BYTES + sizeof(Control) + 1024 <= SMEM_LIMIT, "shared memory over the limit");
    static bool configured[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        e = cudaFuncSetAttribute(gemm_kernel<BN, kTF32, kPair>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kPair ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_kernel<BN, kTF32, kPair>, tm_a, tm_b, tm_c, p);
}

}  // namespace

int gemm_max_resident_pairs(int dtype)
{
    static int cache[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    const int tf = dtype == MPGEMMFI_TF32 ? 1 : 0;
    if (cache[dev][tf] == 0) {
        using C = Cfg<256, true>;
        const size_t smem = (size_t)C::STAGES * C::STAGE_BYTES + OUT_STAGING_BYTES + sizeof(Control) + 1024;
    static_assert(C::STAGES * C::STAGE_BYTES + OUT_STAGING_BYTES + sizeof(Control) + 1024 <= SMEM_LIMIT, "shared memory over the limit");
        auto kern = tf ? gemm_kernel<256, true, true> : gemm_kernel<256, false, true>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2, 1, 1);
        cfg.blockDim = dim3(NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
        cache[dev][tf] = n > 0 ? n : -1;
    }
    return cache[dev][tf] > 0 ? cache[dev][tf] : 0;
}

namespace {
__device__ uint32_t g_launch_slots[LAUNCH_SLOTS][LAUNCH_SLOT_WORDS];
}

namespace {
struct SlotState {
    uint32_t *base = nullptr;            // device address of g_launch_slots
    cudaEvent_t done[LAUNCH_SLOTS] = {};  // recorded behind the last launch that used the slot
    bool used[LAUNCH_SLOTS] = {};
};
SlotState g_slot_state[64];
std::mutex g_slot_mutex;
uint32_t g_launch_counter = 0;
}

cudaError_t gemm_slot_acquire(cudaStream_t stream, int *slot, uint32_t *epoch, uint32_t **signals, uint32_t **ready)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_slot_mutex);
    SlotState &st = g_slot_state[dev];
    if (!st.base) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_launch_slots);
        if (e != cudaSuccess) return e;
        for (int i = 0; i < LAUNCH_SLOTS; ++i) {
            e = cudaEventCreateWithFlags(&st.done[i], cudaEventDisableTiming);
            if (e != cudaSuccess) return e;
        }
        st.base = static_cast<uint32_t *>(ptr);
    }
    const uint32_t n = ++g_launch_counter;
    const int sl = gemm_slot_of(n);
    if (st.used[sl]) {
        // the launch that had this slot LAUNCH_SLOTS launches ago may still be running on another stream
        e = cudaStreamWaitEvent(stream, st.done[sl], 0);
        if (e != cudaSuccess) return e;
    }
    *slot = sl;
    *epoch = gemm_epoch_of(n);
    *signals = st.base + (size_t)sl * LAUNCH_SLOT_WORDS;
    *ready = *signals + SPLIT_SIGNAL_WORDS;
    return cudaSuccess;
}

cudaError_t gemm_slot_release(int slot, cudaStream_t stream)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || slot < 0 || slot >= LAUNCH_SLOTS) return cudaErrorInvalidValue;
    std::lock_guard<std::mutex> lock(g_slot_mutex);
    SlotState &st = g_slot_state[dev];
    e = cudaEventRecord(st.done[slot], stream);
    if (e == cudaSuccess) st.used[slot] = true;
    return e;
}

cudaError_t launch_gemm(int bn, bool pair, const CUtensorMap &tm_a, const CUtensorMap &tm_b, const CUtensorMap &tm_c,
                        const GemmParams &p, int grid, cudaStream_t stream)
{
    const bool tf32 = p.dtype == MPGEMMFI_TF32;
    if (pair)
        return tf32 ? launch_one<256, true, true>(tm_a, tm_b, tm_c, p, grid, stream)
                    : launch_one<256, false, true>(tm_a, tm_b, tm_c, p, grid, stream);
    switch (bn) {
    case 256: return tf32 ? launch_one<256, true, false>(tm_a, tm_b, tm_c, p, grid, stream) : launch_one<256, false, false>(tm_a, tm_b, tm_c, p, grid, stream);
    case 128: return tf32 ? launch_one<128, true, false>(tm_a, tm_b, tm_c, p, grid, stream) : launch_one<128, false, false>(tm_a, tm_b, tm_c, p, grid, stream);
    default:  return tf32 ? launch_one<64, true, false>(tm_a, tm_b, tm_c, p, grid, stream) : launch_one<64, false, false>(tm_a, tm_b, tm_c, p, grid, stream);
    }
}

}  // namespace mpg
