// Grouped GEMMs of the bf16 MoDSE layer on Blackwell tensor cores.
//
// One persistent, warp-specialised kernel template serves the six products of
// the layer (Sec. 3.1, Eq. 4 and its gradient); a tile is 128 rows by up to 256
// fp32 accumulator columns held in tensor memory (TMEM):
//
//   kind            product (per expert e, cp = padded rows, h = width)      K
//   UpGate          Hm = g * silu(xp Wg^T) * (xp Wu^T)      [cp, h]          d
//   Down            o  = Hm Wd_e^T                          [cp, d]  fp32    h
//   DownDgrad       dHm = g * (dyp Wd_e) -> dA, dB          [cp, h]          d
//   DownWgrad       dWd_e = dyp^T Hm                        [d, h]           cp
//   UpGateDgrad     dxp = dA Wg_e + dB Wu_e                 [cp, d]  fp32    2h
//   UpGateWgrad     dWg_e = dA^T xp, dWu_e = dB^T xp        [h, d]           cp
//
// Roles inside a CTA (320 threads): warp 0 issues TMA loads into a 4-stage
// shared-memory ring (every box is 64 elements x 64 rows, 128-byte swizzle),
// warp 1 issues tcgen05.mma with the accumulator in TMEM (two accumulators, so
// the epilogue of one tile overlaps the main loop of the next), warps 2-9 read
// the accumulator with tcgen05.ld (two warps per TMEM lane quadrant, each half
// of the columns) and run the fused epilogue.  Operands are
// consumed either K-major or MN-major straight from their row-major buffers
// (the instruction descriptor carries the major-ness), so the backward pass
// needs no transposed copies.
//
// (g = gate of the row's assignment: it is applied to the hidden row, in fp32,
// before the one rounding to bf16, so neither o nor dY needs a rounded gated
// copy; dyp is dY in group order, bit for bit.)
//
// For backward the up/gate epilogue saves, from its fp32 accumulators A and B,
// sp = B * silu'(A) and sq = silu(A) (bf16): then dA = dHm * sp, dB = dHm * sq, one
// rounded factor each instead of two rounded pre-activations.
//
// Activations that have the hidden axis as their width (Hm, sp, sq, dA, dB)
// are stored as panels: for expert e, panel pc holds
// columns [64 pc, 64 pc + 64) of all cp rows contiguously, so that a single
// two-dimensional tensor map with 128-byte rows describes the whole buffer
// although the row length h differs from expert to expert.
//
// Tiles are handed out statically: experts are ordered by decreasing K so the
// long tiles of wide experts (or of experts with many tokens) start first and
// the short ones fill the tail - the one-GPU form of the paper's expert-pair
// balancing (Sec. 3.2).  Every wait is bounded; a wait that expires records
// kDevTimeout in the status word and the CTA drains and exits.
#include <cuda.h>

#include "tc_gemm.h"

namespace modse {

static int g_force_simt = 0;
static int g_pair_mask = 0;      // bit k: product kind k runs on the two-CTA kernel
// bit k: product kind k runs on the 256-row single-CTA kernel.  Default: the four products with long
// K loops (down, down wgrad, up/gate dgrad, up/gate wgrad), where it measured 4-13 % faster than the
// 128-row kernel; the two products with K = d and heavy epilogues (up/gate, down dgrad) measured slower.
static int g_wide_mask = (1 << 1) | (1 << 3) | (1 << 4) | (1 << 5);
void tc_set_pair_mask(int mask) { g_pair_mask = mask & 63; g_wide_mask = (mask >> 8) & 63; }
int tc_pair_mask() { return g_pair_mask | (g_wide_mask << 8); }

bool tc_force_simt() { return g_force_simt != 0; }
void tc_set_force_simt(int on) { g_force_simt = on ? 1 : 0; }

namespace {

constexpr int kStages = 4;
constexpr int kBoxBytes = 64 * 64 * 2;           // one TMA box: 64 rows of 128 bytes
constexpr int kARegion = 2 * kBoxBytes;          // 128 rows (or 128 MN elements) x 64 K
constexpr int kBRegion = 4 * kBoxBytes;          // up to 256 rows x 64 K
constexpr int kStageBytes = kARegion + kBRegion; // 48 KB
constexpr int kThreads = 320;                   // TMA warp, MMA warp, eight epilogue warps
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait
constexpr int kEpiRowBytes = 64;                 // a 32-element bf16 chunk of one row; 16-byte pieces XOR-swizzled
constexpr int kEpiWarpBytes = 32 * kEpiRowBytes;

struct TcParams {
    LayerMeta meta;
    const int *poffsets;
    const long long *ebase;
    int *status;
    const float *pgate;           // gate of the assignment in each padded row (0 for padding)
    __nv_bfloat16 *hm, *da, *db;
    __nv_bfloat16 *sp, *sq;       // saved for backward: sp = B * silu'(A), sq = silu(A) (panel layout)
    float *o, *dxp;
    __nv_bfloat16 *dw_gate, *dw_up, *dw_down;
    int save;
    int out_f32;   // weight gradients are written as fp32 instead of bf16
};

// dynamic shared memory map (after 1024-byte alignment)
struct SmemTail {
    unsigned char epi_stage[8][kEpiWarpBytes];   // one transposing buffer per epilogue warp
    unsigned long long full[kStages], empty[kStages], tmem_full[2], tmem_empty[2];
    unsigned int tmem_base;
    int abort_flag;
    int order[kMaxExperts];
    int key[kMaxExperts];
    int ntile[kMaxExperts];
    int tstart[kMaxExperts + 1];
};
constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + sizeof(SmemTail);

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false if the phase did not complete within kWaitLimitNs or the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    unsigned it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 255u) == 0) {
            if (*abort_flag || global_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                atomicMax(status, kDevTimeout);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// `nboxes` 64-row boxes stacked from row y on (K-major operand): pairs of them go as one 128-row copy.
__device__ __forceinline__ void tma_load_rows(uint32_t dst, const CUtensorMap *m64, const CUtensorMap *m128, uint32_t bar,
                                              int x, int y, int nboxes)
{
    int i = 0;
    for (; i + 2 <= nboxes; i += 2) tma_load_2d(dst + i * kBoxBytes, m128, bar, x, y + 64 * i);
    if (i < nboxes) tma_load_2d(dst + i * kBoxBytes, m64, bar, x, y + 64 * i);
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), version 1.
//   K-major : rows of 128 bytes, 8-row groups 1024 bytes apart (SBO); LBO unused.
//   MN-major: k-rows of 128 bytes holding 64 MN elements, 8-k groups 1024 bytes
//             apart (SBO), 64-element MN blocks 8192 bytes apart (LBO).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, bool mn_major)
{
    const uint64_t lbo = mn_major ? (uint64_t)(kBoxBytes >> 4) : 1ull;
    const uint64_t sbo = 1024 >> 4;
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128.
__device__ __forceinline__ uint32_t make_idesc(bool a_mn, bool b_mn, int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// Tiles are dealt to the CTAs in rounds of one tile each.  The tile list is sorted by decreasing length of
// the K loop, so within a round the first CTA gets the longest tile; where K is the expert's width (down,
// up/gate dgrad) dealing every round in the same direction hands the same CTAs the longer tile of every
// round (12 % above the mean load for the benchmark's widths), so odd rounds run through the CTAs in
// reverse order, which evens that out (5.5 %, as good as dealing each tile to the least loaded CTA).
// Measured: 4 % on those two products.
template <int KIND>
__device__ __forceinline__ int dealt_tile(int round, int who, int n)
{
    constexpr bool k_varies = (KIND == TcDown || KIND == TcUpGateDgrad);   // K = the expert's width
    return round * n + ((k_varies && (round & 1)) ? n - 1 - who : who);
}

template <int KIND> struct KindTraits;
template <> struct KindTraits<TcUpGate>      { static constexpr bool a_mn = false, b_mn = false; };
template <> struct KindTraits<TcDown>        { static constexpr bool a_mn = false, b_mn = false; };
template <> struct KindTraits<TcDownDgrad>   { static constexpr bool a_mn = false, b_mn = true; };
template <> struct KindTraits<TcDownWgrad>   { static constexpr bool a_mn = true,  b_mn = true; };
template <> struct KindTraits<TcUpGateDgrad> { static constexpr bool a_mn = false, b_mn = true; };
template <> struct KindTraits<TcUpGateWgrad> { static constexpr bool a_mn = true,  b_mn = true; };

// Row block and column block of tile `local` of an expert with mt x nt tiles.
//   N_FASTEST: the column blocks of one row block are consecutive.
//   otherwise: the row blocks of one column block are consecutive, within groups of row blocks that hold at
//   most `rows_per_group` row tiles.  Without the groups an expert with many tokens streams all of its rows
//   once per column block (67 MB of xp per column block at 16 K rows: L2 keeps neither the rows nor the
//   column operand); with them a group's rows stay in L2 while its column blocks go by.  Groups are of
//   equal size (+-1 row tile), so that no group is too small to share the column operand.
template <bool N_FASTEST>
__device__ __forceinline__ void tile_coords(int local, int mt, int nt, int rows_per_group, int &mb, int &nb)
{
    if constexpr (N_FASTEST) {
        mb = local / nt;
        nb = local % nt;
    } else {
        const int n_g = (mt + rows_per_group - 1) / rows_per_group;
        if (n_g <= 1) {
            mb = local % mt;
            nb = local / mt;
            return;
        }
        const int base = mt / n_g, extra = mt % n_g;
        const int big = (base + 1) * nt;              // tiles of each of the first `extra` groups
        int rem, rows, row0;
        if (local < extra * big) {
            const int g = local / big;
            rem = local - g * big; rows = base + 1; row0 = g * (base + 1);
        } else {
            const int l2 = local - extra * big;
            const int g = l2 / (base * nt);
            rem = l2 - g * base * nt; rows = base; row0 = extra * (base + 1) + g * base;
        }
        mb = row0 + rem % rows;
        nb = rem / rows;
    }
}

// Rows of the row operand that one group may hold: 16 M elements (32 MB of bf16) across the model width.
__device__ __forceinline__ int group_row_tiles(int d, int tile_rows) { return max(1, ((16 << 20) / d) / tile_rows); }

struct Tile {
    int e, cp, h, ho, prow0, pbase;   // expert, padded rows, width, width offset, first padded row, first panel row
    int m0, n0, mrows, ncols, nk, which;
    int n_mma, a_boxes, b_boxes;
    int a_boxes_peer, b_off;          // two-CTA tiles only: boxes of the partner's rows, this CTA's column offset
};

// tiles (rows, columns) and K blocks of one expert
template <int KIND>
__device__ __forceinline__ void expert_shape(int cp, int h, int d, int &mt, int &nt, int &nk)
{
    if constexpr (KIND == TcUpGate)      { mt = cp / 128; nt = (h + 127) / 128; nk = d / 64; }
    if constexpr (KIND == TcDown)        { mt = cp / 128; nt = (d + 255) / 256; nk = h / 64; }
    if constexpr (KIND == TcDownDgrad)   { mt = cp / 128; nt = (h + 255) / 256; nk = d / 64; }
    if constexpr (KIND == TcDownWgrad)   { mt = d / 128;  nt = (h + 255) / 256; nk = cp / 64; }
    if constexpr (KIND == TcUpGateDgrad) { mt = cp / 128; nt = (d + 255) / 256; nk = 2 * (h / 64); }
    if constexpr (KIND == TcUpGateWgrad) { mt = 2 * ((h + 127) / 128); nt = (d + 255) / 256; nk = cp / 64; }
}

template <int KIND>
__device__ __forceinline__ Tile decode_tile(const TcParams &prm, const SmemTail *st, int tile, int &cursor)
{
    const int N = prm.meta.N, d = prm.meta.d;
    while (cursor + 1 < N && tile >= st->tstart[cursor + 1]) ++cursor;
    Tile t;
    t.e = st->order[cursor];
    t.ho = prm.meta.hoff[t.e];
    t.h = prm.meta.hoff[t.e + 1] - t.ho;
    t.prow0 = prm.poffsets[t.e];
    t.cp = prm.poffsets[t.e + 1] - t.prow0;
    t.pbase = (int)(prm.ebase[t.e] >> 6);
    int mt, nt, nk;
    expert_shape<KIND>(t.cp, t.h, d, mt, nt, nk);
    const int local = tile - st->tstart[cursor];
    // Order of an expert's tiles (the ~148 tiles in flight should share operands through L2):
    // row-block fastest where the column operand is the big one (weights of the up/gate GEMM, Hm
    // panels of the down wgrad), column-block fastest where all column blocks of one row block
    // fit in flight at once (d / 256 = 8 column blocks), so the row operand is read once.
    constexpr bool n_fastest = (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad);
    int mb, nb;
    tile_coords<n_fastest>(local, mt, nt, group_row_tiles(d, 128), mb, nb);
    t.nk = nk;
    t.which = 0;
    t.mrows = 128;
    if constexpr (KIND == TcUpGate) {
        t.m0 = mb * 128; t.n0 = nb * 128; t.ncols = min(128, t.h - t.n0);
        t.n_mma = 2 * t.ncols; t.a_boxes = 2; t.b_boxes = t.n_mma / 64;
    } else if constexpr (KIND == TcDown || KIND == TcUpGateDgrad) {
        t.m0 = mb * 128; t.n0 = nb * 256; t.ncols = min(256, d - t.n0);
        t.n_mma = t.ncols; t.a_boxes = 2; t.b_boxes = t.ncols / 64;
    } else if constexpr (KIND == TcDownDgrad || KIND == TcDownWgrad) {
        t.m0 = mb * 128; t.n0 = nb * 256; t.ncols = min(256, t.h - t.n0);
        t.n_mma = t.ncols; t.a_boxes = 2; t.b_boxes = t.ncols / 64;
    } else {
        t.which = mb & 1;
        t.m0 = (mb >> 1) * 128; t.n0 = nb * 256; t.ncols = min(256, d - t.n0);
        t.mrows = min(128, t.h - t.m0);
        t.n_mma = t.ncols; t.a_boxes = t.mrows / 64; t.b_boxes = t.ncols / 64;
    }
    return t;
}

// TMA loads of k-block kb of a tile into one stage.
template <int KIND>
__device__ __forceinline__ void issue_loads(const TcMaps &maps, const Tile &t, int kb, uint32_t a_dst, uint32_t b_dst,
                                            uint32_t bar)
{
    if constexpr (KIND == TcUpGate) {
        tma_load_rows(a_dst, &maps.xp, &maps.xp128, bar, kb * 64, t.prow0 + t.m0, 2);
        const int nb = t.ncols / 64;
        tma_load_rows(b_dst, &maps.wgate, &maps.wgate128, bar, kb * 64, t.ho + t.n0, nb);
        tma_load_rows(b_dst + nb * kBoxBytes, &maps.wup, &maps.wup128, bar, kb * 64, t.ho + t.n0, nb);
    } else if constexpr (KIND == TcDown) {
        tma_load_rows(a_dst, &maps.hm, &maps.hm128, bar, 0, t.pbase + kb * t.cp + t.m0, 2);
        tma_load_rows(b_dst, &maps.wdown, &maps.wdown128, bar, t.ho + kb * 64, t.n0, t.b_boxes);
    } else if constexpr (KIND == TcDownDgrad) {
        tma_load_rows(a_dst, &maps.dyp, &maps.dyp128, bar, kb * 64, t.prow0 + t.m0, 2);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d(b_dst + i * kBoxBytes, &maps.wdown, bar, t.ho + t.n0 + 64 * i, kb * 64);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < 2; ++i) tma_load_2d(a_dst + i * kBoxBytes, &maps.dyp, bar, t.m0 + 64 * i, t.prow0 + kb * 64);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d(b_dst + i * kBoxBytes, &maps.hm, bar, 0, t.pbase + (t.n0 / 64 + i) * t.cp + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int half = t.h / 64;
        const bool second = kb >= half;
        const int kk = second ? kb - half : kb;
        const CUtensorMap *bm = second ? &maps.wup : &maps.wgate;
        tma_load_rows(a_dst, second ? &maps.db : &maps.da, second ? &maps.db128 : &maps.da128, bar, 0,
                      t.pbase + kk * t.cp + t.m0, 2);
        for (int i = 0; i < t.b_boxes; ++i) tma_load_2d(b_dst + i * kBoxBytes, bm, bar, t.n0 + 64 * i, t.ho + kk * 64);
    } else {
        const CUtensorMap *am = t.which ? &maps.db : &maps.da;
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d(a_dst + i * kBoxBytes, am, bar, 0, t.pbase + (t.m0 / 64 + i) * t.cp + kb * 64);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d(b_dst + i * kBoxBytes, &maps.xp, bar, t.n0 + 64 * i, t.prow0 + kb * 64);
    }
}

// A warp's 32 threads each hold 32 bf16 values of their own row (64 bytes); the rows are
// `row_stride` elements apart in global memory.  Storing (or loading) them row by row would touch
// 32 lines with 16 bytes each per instruction, so the chunk is transposed through shared memory:
// afterwards four neighbouring lanes cover the 64 bytes of one row and an instruction moves eight
// whole 64-byte row segments.  `own` points at this thread's own row chunk.
// rows_valid: rows of this warp (0..32, counted from the warp's first row) that may be written.
// Byte offset of 16-byte piece q of row r in a warp's staging buffer.  Rows are 64 bytes; the piece index is
// XORed with (r / 2) % 4, so that both access patterns are free of bank conflicts: eight lanes writing the
// same piece of eight consecutive rows, and eight lanes reading all pieces of two consecutive rows.
__device__ __forceinline__ int epi_piece(int r, int q) { return r * kEpiRowBytes + ((q ^ ((r >> 1) & 3)) << 4); }

__device__ __forceinline__ void store_u4x4_staged(unsigned char *stg, int lane, unsigned char *own, long long row_stride_bytes,
                                                  const uint4 (&w)[4], int rows_valid)
{
#pragma unroll
    for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4 *>(stg + epi_piece(lane, q)) = w[q];
    __syncwarp();
    const int q = lane & 3;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int rr = 8 * j + (lane >> 2);
        const uint4 val = *reinterpret_cast<const uint4 *>(stg + epi_piece(rr, q));
        if (rr < rows_valid) *reinterpret_cast<uint4 *>(own + (long long)(rr - lane) * row_stride_bytes + q * 16) = val;
    }
    __syncwarp();
}

__device__ __forceinline__ void store_bf16x32_staged(unsigned char *stg, int lane, __nv_bfloat16 *own, long long row_stride,
                                                     const float (&v)[32], int rows_valid = 32)
{
    uint4 w4[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 t = __floats2bfloat162_rn(v[q * 8 + 2 * i], v[q * 8 + 2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t *>(&t);
        }
        w4[q] = make_uint4(w[0], w[1], w[2], w[3]);
    }
    store_u4x4_staged(stg, lane, reinterpret_cast<unsigned char *>(own), row_stride * 2, w4, rows_valid);
}

// 32 fp32 values per row (128 bytes) go out as two 64-byte halves.
__device__ __forceinline__ void store_f32x32_staged(unsigned char *stg, int lane, float *own, long long row_stride,
                                                    const float (&v)[32], int rows_valid = 32)
{
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        uint4 w4[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            w4[q] = make_uint4(__float_as_uint(v[hh * 16 + 4 * q]), __float_as_uint(v[hh * 16 + 4 * q + 1]),
                               __float_as_uint(v[hh * 16 + 4 * q + 2]), __float_as_uint(v[hh * 16 + 4 * q + 3]));
        store_u4x4_staged(stg, lane, reinterpret_cast<unsigned char *>(own + hh * 16), row_stride * 4, w4, rows_valid);
    }
}

// Transposed (coalesced) load of a warp's 32 row chunks; raw[j] belongs to row 8j + lane/4.
__device__ __forceinline__ void load_bf16x32_transposed(const __nv_bfloat16 *own, long long row_stride, int lane,
                                                        uint4 (&raw)[4])
{
    const int q = lane & 3;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int rr = 8 * j + (lane >> 2);
        raw[j] = *reinterpret_cast<const uint4 *>(own + (long long)(rr - lane) * row_stride + q * 8);
    }
}

// Hands every thread the 64 bytes of its own row out of a transposed load.
__device__ __forceinline__ void untranspose_rows(unsigned char *stg, int lane, const uint4 (&raw)[4], uint4 (&own)[4])
{
    const int q = lane & 3;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int rr = 8 * j + (lane >> 2);
        *reinterpret_cast<uint4 *>(stg + epi_piece(rr, q)) = raw[j];
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) own[i] = *reinterpret_cast<const uint4 *>(stg + epi_piece(lane, i));
    __syncwarp();
}

// Called before the accumulator of a tile is ready: asks L2 for what the epilogue will read from
// global memory (only the down dgrad reads: the two saved SwiGLU factors of its row).
template <int KIND>
__device__ __forceinline__ void epilogue_prefetch(const TcParams &prm, const Tile &t, int row, int c_begin, int c_end)
{
    if constexpr (KIND == TcDownDgrad) {
        for (int c = c_begin; c < c_end; c += 64) {      // one 128-byte line per array covers two 32-column chunks
            const int col = t.n0 + c;
            const size_t idx = ((size_t)(t.pbase + (col >> 6) * t.cp + t.m0 + row) << 6);
            asm volatile("prefetch.global.L2 [%0];" ::"l"(prm.sp + idx));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(prm.sq + idx));
        }
    }
}

// Epilogue of one tile for one thread: accumulator row `row`, columns [c_begin, c_end).
template <int KIND>
__device__ __forceinline__ void epilogue_row(const TcParams &prm, const Tile &t, uint32_t tacc, int row, int c_begin,
                                             int c_end, unsigned char *stg)
{
    const int lane = row & 31;
    const int d = prm.meta.d, S = prm.meta.S;
    const bool have_acc = t.nk > 0;
    auto panel_index = [&](int c) {
        const int col = t.n0 + c;
        return ((size_t)(t.pbase + (col >> 6) * t.cp + t.m0 + row) << 6) + (col & 63);
    };
    if constexpr (KIND == TcUpGate) {
        const float gate = prm.pgate[t.prow0 + t.m0 + row];
        for (int c = c_begin; c < c_end; c += 32) {
            uint32_t ra[32], rb[32];
            tmem_ld32(tacc + c, ra);
            tmem_ld32(tacc + t.ncols + c, rb);
            tmem_ld_wait();
            const size_t idx = panel_index(c);
            float hm[32];
            if (prm.save) {
                float sp[32], sq[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float av = __uint_as_float(ra[i]), bv = __uint_as_float(rb[i]);
                    const float sg = __fdividef(1.0f, 1.0f + __expf(-av));   // ex2 + rcp: a full-precision division here slows the MMA warp
                    sq[i] = av * sg;
                    sp[i] = bv * sg * (1.0f + av * (1.0f - sg));
                    hm[i] = gate * (sq[i] * bv);
                }
                store_bf16x32_staged(stg, lane, prm.sp + idx, 64, sp);
                store_bf16x32_staged(stg, lane, prm.sq + idx, 64, sq);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const float av = __uint_as_float(ra[i]), bv = __uint_as_float(rb[i]);
                    hm[i] = gate * (av * __fdividef(1.0f, 1.0f + __expf(-av)) * bv);
                }
            }
            store_bf16x32_staged(stg, lane, prm.hm + idx, 64, hm);
        }
    } else if constexpr (KIND == TcDown || KIND == TcUpGateDgrad) {
        float *out = (KIND == TcDown ? prm.o : prm.dxp) + (size_t)(t.prow0 + t.m0 + row) * d + t.n0;
        for (int c = c_begin; c < c_end; c += 32) {
            uint32_t r[32];
            float v[32];
            tmem_ld32(tacc + c, r);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
            store_f32x32_staged(stg, lane, out + c, d, v);
        }
    } else if constexpr (KIND == TcDownDgrad) {
        // dA = dHm * sp, dB = dHm * sq with dHm = gate * acc; the saved factors of the next
        // chunk are fetched while this one is computed
        const float gate = prm.pgate[t.prow0 + t.m0 + row];
        uint4 praw[4], qraw[4];            // transposed: entry j belongs to row 8j + lane/4 of this warp
        {
            const size_t idx = panel_index(c_begin);
            load_bf16x32_transposed(prm.sp + idx, 64, lane, praw);
            load_bf16x32_transposed(prm.sq + idx, 64, lane, qraw);
        }
        for (int c = c_begin; c < c_end; c += 32) {
            uint32_t r[32];
            tmem_ld32(tacc + c, r);
            uint4 pn[4], qn[4];
            const bool more = c + 32 < c_end;
            if (more) {
                const size_t nidx = panel_index(c + 32);
                load_bf16x32_transposed(prm.sp + nidx, 64, lane, pn);
                load_bf16x32_transposed(prm.sq + nidx, 64, lane, qn);
            }
            uint4 pown[4], qown[4];
            untranspose_rows(stg, lane, praw, pown);
            untranspose_rows(stg, lane, qraw, qown);
            tmem_ld_wait();
            const size_t idx = panel_index(c);
            float da[32], db[32];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const uint32_t pw[4] = {pown[q4].x, pown[q4].y, pown[q4].z, pown[q4].w};
                const uint32_t qw[4] = {qown[q4].x, qown[q4].y, qown[q4].z, qown[q4].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int e0 = q4 * 8 + 2 * i;
                    const float dh0 = gate * __uint_as_float(r[e0]), dh1 = gate * __uint_as_float(r[e0 + 1]);
                    da[e0] = dh0 * __uint_as_float(pw[i] << 16);
                    da[e0 + 1] = dh1 * __uint_as_float(pw[i] & 0xFFFF0000u);
                    db[e0] = dh0 * __uint_as_float(qw[i] << 16);
                    db[e0 + 1] = dh1 * __uint_as_float(qw[i] & 0xFFFF0000u);
                }
            }
            store_bf16x32_staged(stg, lane, prm.da + idx, 64, da);
            store_bf16x32_staged(stg, lane, prm.db + idx, 64, db);
            if (more) {
#pragma unroll
                for (int i = 0; i < 4; ++i) { praw[i] = pn[i]; qraw[i] = qn[i]; }
            }
        }
    } else if constexpr (KIND == TcDownWgrad) {
        const size_t oidx = (size_t)(t.m0 + row) * S + t.ho + t.n0;
        for (int c = c_begin; c < c_end; c += 32) {
            float v[32];
            if (have_acc) {
                uint32_t r[32];
                tmem_ld32(tacc + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0.f;
            }
            if (prm.out_f32) store_f32x32_staged(stg, lane, reinterpret_cast<float *>(prm.dw_down) + oidx + c, S, v);
            else store_bf16x32_staged(stg, lane, prm.dw_down + oidx + c, S, v);
        }
    } else {
        __nv_bfloat16 *obase = t.which ? prm.dw_up : prm.dw_gate;
        const size_t oidx = (size_t)(t.ho + t.m0 + row) * d + t.n0;
        for (int c = c_begin; c < c_end; c += 32) {
            float v[32];
            if (have_acc) {
                uint32_t r[32];
                tmem_ld32(tacc + c, r);      // whole warp takes part in the load, also for rows that are not stored
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0.f;
            }
            const int rows_valid = t.mrows - (row - lane);      // rows of this warp inside the expert's width
            if (prm.out_f32) store_f32x32_staged(stg, lane, reinterpret_cast<float *>(obase) + oidx + c, d, v, rows_valid);
            else store_bf16x32_staged(stg, lane, obase + oidx + c, d, v, rows_valid);
        }
    }
}

template <int KIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_grouped_gemm(const __grid_constant__ TcMaps maps, const __grid_constant__ TcParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    unsigned char *smem = smem_raw + pad;
    const uint32_t stage_base = raw + pad;
    SmemTail *st = reinterpret_cast<SmemTail *>(smem + (size_t)kStages * kStageBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = prm.meta.N, d = prm.meta.d;

    // ---- schedule: experts by decreasing K, tiles of an expert contiguous ----
    for (int e = tid; e < N; e += kThreads) {
        const int cp = prm.poffsets[e + 1] - prm.poffsets[e];
        const int h = prm.meta.hoff[e + 1] - prm.meta.hoff[e];
        int mt, nt, nk;
        expert_shape<KIND>(cp, h, d, mt, nt, nk);
        st->ntile[e] = mt * nt;
        st->key[e] = nk;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&st->full[s]), 1);
            mbar_init(smem_u32(&st->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&st->tmem_full[a]), 1);
            mbar_init(smem_u32(&st->tmem_empty[a]), 256);
        }
        st->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    for (int e = tid; e < N; e += kThreads) {
        int rank = 0;
        const int ke = st->key[e];
        for (int f = 0; f < N; ++f) {
            const int kf = st->key[f];
            rank += (kf > ke) || (kf == ke && f < e);
        }
        st->order[rank] = e;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&st->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int i = 0; i < N; ++i) { st->tstart[i] = acc; acc += st->ntile[st->order[i]]; }
        st->tstart[N] = acc;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = st->tmem_base;
    const int total_tiles = st->tstart[N];
    volatile int *abort_flag = &st->abort_flag;

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x)) {
                const Tile t = decode_tile<KIND>(prm, st, tile, cursor);
                const uint32_t bytes = (uint32_t)(t.a_boxes + t.b_boxes) * kBoxBytes;
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&st->full[stage]);
                    mbar_arrive_expect_tx(bar, bytes);
                    const uint32_t a_dst = stage_base + stage * kStageBytes;
                    issue_loads<KIND>(maps, t, kb, a_dst, a_dst + kARegion, bar);
                    ++issued;
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA leaves: wait (bounded) for
                // the current phase of every stage that has had a load
                const int n = issued < kStages ? (int)issued : kStages;
                for (int i = 1; i <= n; ++i) {
                    int s = stage - i;
                    uint32_t ph = phase;
                    if (s < 0) { s += kStages; ph ^= 1u; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(smem_u32(&st->full[s]), ph) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            int stage = 0, cursor = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            constexpr bool a_mn = KindTraits<KIND>::a_mn, b_mn = KindTraits<KIND>::b_mn;
            constexpr uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
            constexpr uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
            for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x), ++it) {
                const Tile t = decode_tile<KIND>(prm, st, tile, cursor);
                const int acc = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(acc * kAccCols);
                const uint32_t idesc = make_idesc(a_mn, b_mn, t.n_mma);
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->full[stage]), phase, abort_flag, prm.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage_base + stage * kStageBytes;
                    const uint64_t adesc = make_desc(a_addr, a_mn);
                    const uint64_t bdesc = make_desc(a_addr + kARegion, b_mn);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16(tacc, adesc + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step), idesc,
                                  (kb > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(smem_u32(&st->empty[stage]));   // frees the stage once these MMAs have read it
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (t.nk > 0) umma_commit(smem_u32(&st->tmem_full[acc]));
                else mbar_arrive(smem_u32(&st->tmem_full[acc]));
            }
        }
    } else {
        // ===================== epilogue (warps 2..9) =====================
        const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;          // which half of the tile's columns
        const int row = quad * 32 + lane;
        int cursor = 0, it = 0;
        bool ok = true;
        for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x), ++it) {
            const Tile t = decode_tile<KIND>(prm, st, tile, cursor);
            const int acc = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            const int chalf = t.ncols >> 1;            // a multiple of 32: ncols is a multiple of 64
            epilogue_prefetch<KIND>(prm, t, row, half * chalf, (half + 1) * chalf);
            if (!mbar_wait(smem_u32(&st->tmem_full[acc]), acc_phase, abort_flag, prm.status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccCols);
            epilogue_row<KIND>(prm, t, tacc, row, half * chalf, (half + 1) * chalf, st->epi_stage[warp - 2]);
            tc_fence_before();
            mbar_arrive(smem_u32(&st->tmem_empty[acc]));
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ===========================================================================
// Two-CTA variant (cta_group::2).  A cluster of two CTAs on neighbouring SMs
// computes one 256-row tile: each CTA stages its own 128 rows of the row
// operand and HALF of the column operand (so a CTA moves 32 KB per k-block
// instead of 48 KB), the leader CTA (cluster rank 0) issues tcgen05.mma with
// M = 256 reading both CTAs' shared memory, and each CTA's TMEM receives the
// accumulator rows of its own half.  Barrier protocol:
//   full[s]       leader only; its producer posts the byte count of both CTAs,
//                 both producers' TMA loads complete on it
//   empty[s]      one per CTA; tcgen05.commit multicasts to both
//   tmem_full[a]  one per CTA; tcgen05.commit multicasts to both
//   tmem_empty[a] leader only; one arrival per epilogue warp of both CTAs
// ===========================================================================
constexpr int kStages2 = 6;
constexpr int kARegion2 = 2 * kBoxBytes;
constexpr int kBRegion2 = 2 * kBoxBytes;
constexpr int kStageBytes2 = kARegion2 + kBRegion2;   // 32 KB
struct SmemTail2 {
    unsigned char epi_stage[8][kEpiWarpBytes];   // one transposing buffer per epilogue warp
    unsigned long long full[kStages2], empty[kStages2], tmem_full[2], tmem_empty[2];
    unsigned int tmem_base;
    int abort_flag;
    int order[kMaxExperts];
    int key[kMaxExperts];
    int ntile[kMaxExperts];
    int tstart[kMaxExperts + 1];
};
constexpr size_t kSmemBytes2 = 1024 + (size_t)kStages2 * kStageBytes2 + sizeof(SmemTail2);

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t leader_bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(leader_bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
__device__ __forceinline__ uint32_t make_idesc_pair(bool a_mn, bool b_mn, int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

template <int KIND>
__device__ __forceinline__ void expert_shape2(int cp, int h, int d, int &mt, int &nt, int &nk)
{
    if constexpr (KIND == TcUpGate)      { mt = (cp + 255) / 256; nt = (h + 127) / 128; nk = d / 64; }
    if constexpr (KIND == TcDown)        { mt = (cp + 255) / 256; nt = (d + 255) / 256; nk = h / 64; }
    if constexpr (KIND == TcDownDgrad)   { mt = (cp + 255) / 256; nt = (h + 255) / 256; nk = d / 64; }
    if constexpr (KIND == TcDownWgrad)   { mt = (d + 255) / 256;  nt = (h + 255) / 256; nk = cp / 64; }
    if constexpr (KIND == TcUpGateDgrad) { mt = (cp + 255) / 256; nt = (d + 255) / 256; nk = 2 * (h / 64); }
    if constexpr (KIND == TcUpGateWgrad) { mt = 2 * ((h + 255) / 256); nt = (d + 255) / 256; nk = cp / 64; }
}

// Tile of this CTA (cluster rank `rank`) inside pair tile `tile`.  Fields as in the one-CTA
// decode; m0 / mrows / a_boxes describe this CTA's 128-row half, a_boxes_peer the other half,
// b_boxes and b_off this CTA's half of the column operand, ncols the columns that are stored.
template <int KIND>
__device__ __forceinline__ Tile decode_tile2(const TcParams &prm, const SmemTail2 *st, int tile, int &cursor, int rank)
{
    const int N = prm.meta.N, d = prm.meta.d;
    while (cursor + 1 < N && tile >= st->tstart[cursor + 1]) ++cursor;
    Tile t;
    t.e = st->order[cursor];
    t.ho = prm.meta.hoff[t.e];
    t.h = prm.meta.hoff[t.e + 1] - t.ho;
    t.prow0 = prm.poffsets[t.e];
    t.cp = prm.poffsets[t.e + 1] - t.prow0;
    t.pbase = (int)(prm.ebase[t.e] >> 6);
    int mt, nt, nk;
    expert_shape2<KIND>(t.cp, t.h, d, mt, nt, nk);
    const int local = tile - st->tstart[cursor];
    constexpr bool n_fastest = (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad);
    int mb, nb;
    tile_coords<n_fastest>(local, mt, nt, group_row_tiles(d, 256), mb, nb);
    t.nk = nk;
    t.which = 0;
    int row_extent;                       // extent of the tile's row dimension for this expert
    if constexpr (KIND == TcDownWgrad) row_extent = d;
    else if constexpr (KIND == TcUpGateWgrad) { row_extent = t.h; t.which = mb & 1; mb >>= 1; }
    else row_extent = t.cp;
    const int m_pair = mb * 256;
    t.m0 = m_pair + 128 * rank;
    t.mrows = max(0, min(128, row_extent - t.m0));
    const int peer_rows = max(0, min(128, row_extent - (m_pair + 128 * (1 - rank))));
    t.a_boxes = t.mrows / 64;
    t.a_boxes_peer = peer_rows / 64;
    if constexpr (KIND == TcUpGate) {
        t.n0 = nb * 128; t.ncols = min(128, t.h - t.n0);
        t.n_mma = 2 * t.ncols; t.b_boxes = t.ncols / 64; t.b_off = 0;
    } else if constexpr (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad) {
        t.n0 = nb * 256; t.ncols = min(256, d - t.n0);
        t.n_mma = t.ncols; t.b_boxes = t.ncols / 128; t.b_off = rank * (t.ncols / 2);
    } else {
        t.n0 = nb * 256; t.ncols = min(256, t.h - t.n0);
        t.n_mma = (t.ncols + 127) & ~127; t.b_boxes = t.n_mma / 128; t.b_off = rank * (t.n_mma / 2);
    }
    return t;
}

template <int KIND>
__device__ __forceinline__ void issue_loads2(const TcMaps &maps, const Tile &t, int rank, int kb, uint32_t a_dst,
                                             uint32_t b_dst, uint32_t bar)
{
    if constexpr (KIND == TcUpGate) {
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, &maps.xp, bar, kb * 64, t.prow0 + t.m0 + 64 * i);
        const CUtensorMap *bm = rank ? &maps.wup : &maps.wgate;     // gate columns live in CTA 0, up columns in CTA 1
        for (int i = 0; i < t.b_boxes; ++i) tma_load_2d_pair(b_dst + i * kBoxBytes, bm, bar, kb * 64, t.ho + t.n0 + 64 * i);
    } else if constexpr (KIND == TcDown) {
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, &maps.hm, bar, 0, t.pbase + kb * t.cp + t.m0 + 64 * i);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d_pair(b_dst + i * kBoxBytes, &maps.wdown, bar, t.ho + kb * 64, t.n0 + t.b_off + 64 * i);
    } else if constexpr (KIND == TcDownDgrad) {
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, &maps.dyp, bar, kb * 64, t.prow0 + t.m0 + 64 * i);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d_pair(b_dst + i * kBoxBytes, &maps.wdown, bar, t.ho + t.n0 + t.b_off + 64 * i, kb * 64);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, &maps.dyp, bar, t.m0 + 64 * i, t.prow0 + kb * 64);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d_pair(b_dst + i * kBoxBytes, &maps.hm, bar, 0,
                             t.pbase + ((t.n0 + t.b_off) / 64 + i) * t.cp + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int half = t.h / 64;
        const bool second = kb >= half;
        const int kk = second ? kb - half : kb;
        const CUtensorMap *am = second ? &maps.db : &maps.da;
        const CUtensorMap *bm = second ? &maps.wup : &maps.wgate;
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, am, bar, 0, t.pbase + kk * t.cp + t.m0 + 64 * i);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d_pair(b_dst + i * kBoxBytes, bm, bar, t.n0 + t.b_off + 64 * i, t.ho + kk * 64);
    } else {
        const CUtensorMap *am = t.which ? &maps.db : &maps.da;
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(a_dst + i * kBoxBytes, am, bar, 0, t.pbase + (t.m0 / 64 + i) * t.cp + kb * 64);
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d_pair(b_dst + i * kBoxBytes, &maps.xp, bar, t.n0 + t.b_off + 64 * i, t.prow0 + kb * 64);
    }
}

template <int KIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_grouped_gemm_pair(const __grid_constant__ TcMaps maps, const __grid_constant__ TcParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    unsigned char *smem = smem_raw + pad;
    const uint32_t stage_base = raw + pad;
    SmemTail2 *st = reinterpret_cast<SmemTail2 *>(smem + (size_t)kStages2 * kStageBytes2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = prm.meta.N, d = prm.meta.d;
    const int rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    for (int e = tid; e < N; e += kThreads) {
        const int cp = prm.poffsets[e + 1] - prm.poffsets[e];
        const int h = prm.meta.hoff[e + 1] - prm.meta.hoff[e];
        int mt, nt, nk;
        expert_shape2<KIND>(cp, h, d, mt, nt, nk);
        st->ntile[e] = mt * nt;
        st->key[e] = nk;
    }
    if (tid == 0) {
        for (int s = 0; s < kStages2; ++s) {
            mbar_init(smem_u32(&st->full[s]), 1);
            mbar_init(smem_u32(&st->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&st->tmem_full[a]), 1);
            mbar_init(smem_u32(&st->tmem_empty[a]), 16);      // 8 epilogue warps of each of the two CTAs
        }
        st->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    for (int e = tid; e < N; e += kThreads) {
        int rk = 0;
        const int ke = st->key[e];
        for (int f = 0; f < N; ++f) {
            const int kf = st->key[f];
            rk += (kf > ke) || (kf == ke && f < e);
        }
        st->order[rk] = e;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&st->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int i = 0; i < N; ++i) { st->tstart[i] = acc; acc += st->ntile[st->order[i]]; }
        st->tstart[N] = acc;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // both CTAs' barriers exist before any remote arrive or TMA completion
    tc_fence_after();
    const uint32_t tmem_base = st->tmem_base;
    const int total_tiles = st->tstart[N];
    volatile int *abort_flag = &st->abort_flag;

    if (warp == 0) {
        // ===================== TMA producer (both CTAs) =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int rnd = 0, tile = dealt_tile<KIND>(0, cluster_id, n_clusters); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, cluster_id, n_clusters)) {
                const Tile t = decode_tile2<KIND>(prm, st, tile, cursor, rank);
                const uint32_t bytes = (uint32_t)(t.a_boxes + t.a_boxes_peer + 2 * t.b_boxes) * kBoxBytes;
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                    const uint32_t leader_bar = map_to_cta(smem_u32(&st->full[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&st->full[stage]), bytes);
                    const uint32_t a_dst = stage_base + stage * kStageBytes2;
                    issue_loads2<KIND>(maps, t, rank, kb, a_dst, a_dst + kARegion2, leader_bar);
                    ++issued;
                    if (++stage == kStages2) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok && rank == 0) {
                const int n = issued < kStages2 ? (int)issued : kStages2;
                for (int i = 1; i <= n; ++i) {
                    int s = stage - i;
                    uint32_t ph = phase;
                    if (s < 0) { s += kStages2; ph ^= 1u; }
                    const unsigned long long t0 = global_ns();
                    while (!mbar_try_wait(smem_u32(&st->full[s]), ph) && global_ns() - t0 < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer (leader CTA only) =====================
        if (lane == 0 && rank == 0) {
            int stage = 0, cursor = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            constexpr bool a_mn = KindTraits<KIND>::a_mn, b_mn = KindTraits<KIND>::b_mn;
            constexpr uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
            constexpr uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
            for (int rnd = 0, tile = dealt_tile<KIND>(0, cluster_id, n_clusters); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, cluster_id, n_clusters), ++it) {
                const Tile t = decode_tile2<KIND>(prm, st, tile, cursor, 0);
                const int acc = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(acc * kAccCols);
                const uint32_t idesc = make_idesc_pair(a_mn, b_mn, t.n_mma);
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->full[stage]), phase, abort_flag, prm.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage_base + stage * kStageBytes2;
                    const uint64_t adesc = make_desc(a_addr, a_mn);
                    const uint64_t bdesc = make_desc(a_addr + kARegion2, b_mn);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_pair(tacc, adesc + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step), idesc,
                                       (kb > 0 || ks > 0) ? 1u : 0u);
                    umma_commit_pair(smem_u32(&st->empty[stage]));
                    if (++stage == kStages2) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (t.nk > 0) {
                    umma_commit_pair(smem_u32(&st->tmem_full[acc]));
                } else {
                    mbar_arrive(smem_u32(&st->tmem_full[acc]));
                    mbar_arrive_cluster(map_to_cta(smem_u32(&st->tmem_full[acc]), 1));
                }
            }
        }
    } else {
        // ===================== epilogue (warps 2..9, both CTAs) =====================
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row = quad * 32 + lane;
        int cursor = 0, it = 0;
        bool ok = true;
        for (int rnd = 0, tile = dealt_tile<KIND>(0, cluster_id, n_clusters); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, cluster_id, n_clusters), ++it) {
            const Tile t = decode_tile2<KIND>(prm, st, tile, cursor, rank);
            const int acc = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            if (!mbar_wait(smem_u32(&st->tmem_full[acc]), acc_phase, abort_flag, prm.status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccCols);
            if (t.mrows > 0) {
                // split the accumulator columns between the two warps of a lane quadrant, store only valid ones
                const int span = (KIND == TcUpGate) ? t.ncols : t.n_mma;
                const int chalf = span >> 1;
                const int c0 = half * chalf, c1 = min((half + 1) * chalf, t.ncols);
                if (c0 < c1) epilogue_row<KIND>(prm, t, tacc, row, c0, c1, st->epi_stage[warp - 2]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (rank == 0) mbar_arrive(smem_u32(&st->tmem_empty[acc]));
                else mbar_arrive_cluster(map_to_cta(smem_u32(&st->tmem_empty[acc]), 0));
            }
        }
    }

    // ---- teardown: nobody leaves while its partner may still touch its shared or tensor memory ----
    tc_fence_before();
    __syncthreads();
    __syncwarp();
    cluster_sync_all();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ===========================================================================
// Wide variant: one CTA computes a 256-row tile as two 128-row halves that
// share the column operand.  A k-block then stages 32 KB of rows + 32 KB of
// columns for twice the MMA work of the 128-row kernel, i.e. 2/3 of the bytes
// per FLOP through L2 -> shared memory, which is what bounds the 128-row
// kernel (it needs ~19.5 TB/s of L2 reads at the MMA rate; the path saturates
// near 22 TB/s).  The price: both accumulators (2 x 256 TMEM columns) belong
// to the current tile, so the epilogue of a tile overlaps only the part of the
// next tile's main loop that does not touch the half being drained.  Used for
// the products with long K loops, where that exposure is a few percent.
// ===========================================================================
constexpr int kStagesW = 3;
constexpr int kARegionW = 4 * kBoxBytes;            // two halves of 128 rows x 64 K
constexpr int kStageBytesW = kARegionW + kBRegion;  // 64 KB
struct SmemTailW {
    unsigned char epi_stage[8][kEpiWarpBytes];   // one transposing buffer per epilogue warp
    unsigned long long full[kStagesW], empty[kStagesW], tmem_full[1], tmem_empty[2];
    unsigned int tmem_base;
    int abort_flag;
    int order[kMaxExperts];
    int key[kMaxExperts];
    int ntile[kMaxExperts];
    int tstart[kMaxExperts + 1];
};
constexpr size_t kSmemBytesW = 1024 + (size_t)kStagesW * kStageBytesW + sizeof(SmemTailW);

template <int KIND>
__device__ __forceinline__ void expert_shape_wide(int cp, int h, int d, int &mt, int &nt, int &nk)
{
    if constexpr (KIND == TcUpGate)      { mt = (cp + 255) / 256; nt = (h + 127) / 128; nk = d / 64; }
    if constexpr (KIND == TcDown)        { mt = (cp + 255) / 256; nt = (d + 255) / 256; nk = h / 64; }
    if constexpr (KIND == TcDownDgrad)   { mt = (cp + 255) / 256; nt = (h + 255) / 256; nk = d / 64; }
    if constexpr (KIND == TcDownWgrad)   { mt = (d + 255) / 256;  nt = (h + 255) / 256; nk = cp / 64; }
    if constexpr (KIND == TcUpGateDgrad) { mt = (cp + 255) / 256; nt = (d + 255) / 256; nk = 2 * (h / 64); }
    if constexpr (KIND == TcUpGateWgrad) { mt = 2 * ((h + 255) / 256); nt = (d + 255) / 256; nk = cp / 64; }
}

// First half (rows m0 .. m0+127) of wide tile `tile`; a_boxes_peer carries the second half's boxes.
template <int KIND>
__device__ __forceinline__ Tile decode_tile_wide(const TcParams &prm, const SmemTailW *st, int tile, int &cursor)
{
    const int N = prm.meta.N, d = prm.meta.d;
    while (cursor + 1 < N && tile >= st->tstart[cursor + 1]) ++cursor;
    Tile t;
    t.e = st->order[cursor];
    t.ho = prm.meta.hoff[t.e];
    t.h = prm.meta.hoff[t.e + 1] - t.ho;
    t.prow0 = prm.poffsets[t.e];
    t.cp = prm.poffsets[t.e + 1] - t.prow0;
    t.pbase = (int)(prm.ebase[t.e] >> 6);
    int mt, nt, nk;
    expert_shape_wide<KIND>(t.cp, t.h, d, mt, nt, nk);
    const int local = tile - st->tstart[cursor];
    constexpr bool n_fastest = (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad);
    int mb, nb;
    tile_coords<n_fastest>(local, mt, nt, group_row_tiles(d, 256), mb, nb);
    t.nk = nk;
    t.which = 0;
    int row_extent;
    if constexpr (KIND == TcDownWgrad) row_extent = d;
    else if constexpr (KIND == TcUpGateWgrad) { row_extent = t.h; t.which = mb & 1; mb >>= 1; }
    else row_extent = t.cp;
    t.m0 = mb * 256;
    t.mrows = max(0, min(128, row_extent - t.m0));
    t.a_boxes = t.mrows / 64;
    t.a_boxes_peer = max(0, min(128, row_extent - t.m0 - 128)) / 64;
    t.b_off = 0;
    if constexpr (KIND == TcUpGate) {
        t.n0 = nb * 128; t.ncols = min(128, t.h - t.n0);
        t.n_mma = 2 * t.ncols; t.b_boxes = t.n_mma / 64;
    } else if constexpr (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad) {
        t.n0 = nb * 256; t.ncols = min(256, d - t.n0);
        t.n_mma = t.ncols; t.b_boxes = t.ncols / 64;
    } else {
        t.n0 = nb * 256; t.ncols = min(256, t.h - t.n0);
        t.n_mma = t.ncols; t.b_boxes = t.ncols / 64;
    }
    return t;
}

__device__ __forceinline__ Tile second_half(const Tile &t)
{
    Tile u = t;
    u.m0 = t.m0 + 128;
    u.a_boxes = t.a_boxes_peer;
    u.mrows = 64 * t.a_boxes_peer;
    return u;
}

// Row-operand boxes of one 128-row half.
template <int KIND>
__device__ __forceinline__ void load_rows(const TcMaps &maps, const Tile &t, int kb, uint32_t dst, uint32_t bar)
{
    if constexpr (KIND == TcUpGate) {
        tma_load_rows(dst, &maps.xp, &maps.xp128, bar, kb * 64, t.prow0 + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDown) {
        tma_load_rows(dst, &maps.hm, &maps.hm128, bar, 0, t.pbase + kb * t.cp + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDownDgrad) {
        tma_load_rows(dst, &maps.dyp, &maps.dyp128, bar, kb * 64, t.prow0 + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < t.a_boxes; ++i) tma_load_2d(dst + i * kBoxBytes, &maps.dyp, bar, t.m0 + 64 * i, t.prow0 + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int half = t.h / 64;
        const bool second = kb >= half;
        const int kk = second ? kb - half : kb;
        tma_load_rows(dst, second ? &maps.db : &maps.da, second ? &maps.db128 : &maps.da128, bar, 0,
                      t.pbase + kk * t.cp + t.m0, t.a_boxes);
    } else {
        const CUtensorMap *am = t.which ? &maps.db : &maps.da;
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d(dst + i * kBoxBytes, am, bar, 0, t.pbase + (t.m0 / 64 + i) * t.cp + kb * 64);
    }
}

// Column-operand boxes of a tile.
template <int KIND>
__device__ __forceinline__ void load_cols(const TcMaps &maps, const Tile &t, int kb, uint32_t dst, uint32_t bar)
{
    if constexpr (KIND == TcUpGate) {
        const int nb = t.ncols / 64;
        tma_load_rows(dst, &maps.wgate, &maps.wgate128, bar, kb * 64, t.ho + t.n0, nb);
        tma_load_rows(dst + nb * kBoxBytes, &maps.wup, &maps.wup128, bar, kb * 64, t.ho + t.n0, nb);
    } else if constexpr (KIND == TcDown) {
        tma_load_rows(dst, &maps.wdown, &maps.wdown128, bar, t.ho + kb * 64, t.n0, t.b_boxes);
    } else if constexpr (KIND == TcDownDgrad) {
        for (int i = 0; i < t.b_boxes; ++i) tma_load_2d(dst + i * kBoxBytes, &maps.wdown, bar, t.ho + t.n0 + 64 * i, kb * 64);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < t.b_boxes; ++i)
            tma_load_2d(dst + i * kBoxBytes, &maps.hm, bar, 0, t.pbase + (t.n0 / 64 + i) * t.cp + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int half = t.h / 64;
        const bool second = kb >= half;
        const int kk = second ? kb - half : kb;
        const CUtensorMap *bm = second ? &maps.wup : &maps.wgate;
        for (int i = 0; i < t.b_boxes; ++i) tma_load_2d(dst + i * kBoxBytes, bm, bar, t.n0 + 64 * i, t.ho + kk * 64);
    } else {
        for (int i = 0; i < t.b_boxes; ++i) tma_load_2d(dst + i * kBoxBytes, &maps.xp, bar, t.n0 + 64 * i, t.prow0 + kb * 64);
    }
}

template <int KIND>
__global__ void __launch_bounds__(kThreads, 1)
tc_grouped_gemm_wide(const __grid_constant__ TcMaps maps, const __grid_constant__ TcParams prm)
{
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    unsigned char *smem = smem_raw + pad;
    const uint32_t stage_base = raw + pad;
    SmemTailW *st = reinterpret_cast<SmemTailW *>(smem + (size_t)kStagesW * kStageBytesW);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int N = prm.meta.N, d = prm.meta.d;

    for (int e = tid; e < N; e += kThreads) {
        const int cp = prm.poffsets[e + 1] - prm.poffsets[e];
        const int h = prm.meta.hoff[e + 1] - prm.meta.hoff[e];
        int mt, nt, nk;
        expert_shape_wide<KIND>(cp, h, d, mt, nt, nk);
        st->ntile[e] = mt * nt;
        st->key[e] = nk;
    }
    if (tid == 0) {
        for (int s = 0; s < kStagesW; ++s) {
            mbar_init(smem_u32(&st->full[s]), 1);
            mbar_init(smem_u32(&st->empty[s]), 1);
        }
        mbar_init(smem_u32(&st->tmem_full[0]), 1);
        mbar_init(smem_u32(&st->tmem_empty[0]), 256);
        mbar_init(smem_u32(&st->tmem_empty[1]), 256);
        st->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    for (int e = tid; e < N; e += kThreads) {
        int rk = 0;
        const int ke = st->key[e];
        for (int f = 0; f < N; ++f) {
            const int kf = st->key[f];
            rk += (kf > ke) || (kf == ke && f < e);
        }
        st->order[rk] = e;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&st->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int i = 0; i < N; ++i) { st->tstart[i] = acc; acc += st->ntile[st->order[i]]; }
        st->tstart[N] = acc;
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = st->tmem_base;
    const int total_tiles = st->tstart[N];
    volatile int *abort_flag = &st->abort_flag;

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x)) {
                const Tile t0 = decode_tile_wide<KIND>(prm, st, tile, cursor);
                const Tile t1 = second_half(t0);
                const uint32_t bytes = (uint32_t)(t0.a_boxes + t1.a_boxes + t0.b_boxes) * kBoxBytes;
                for (int kb = 0; kb < t0.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->empty[stage]), phase ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                    const uint32_t bar = smem_u32(&st->full[stage]);
                    mbar_arrive_expect_tx(bar, bytes);
                    const uint32_t a_dst = stage_base + stage * kStageBytesW;
                    load_rows<KIND>(maps, t0, kb, a_dst, bar);
                    load_rows<KIND>(maps, t1, kb, a_dst + kARegion, bar);
                    load_cols<KIND>(maps, t0, kb, a_dst + kARegionW, bar);
                    ++issued;
                    if (++stage == kStagesW) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                const int n = issued < kStagesW ? (int)issued : kStagesW;
                for (int i = 1; i <= n; ++i) {
                    int s = stage - i;
                    uint32_t ph = phase;
                    if (s < 0) { s += kStagesW; ph ^= 1u; }
                    const unsigned long long tb = global_ns();
                    while (!mbar_try_wait(smem_u32(&st->full[s]), ph) && global_ns() - tb < kWaitLimitNs) {}
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            uint32_t use0 = 0, use1 = 0;         // how often each accumulator has been handed to the epilogue
            bool ok = true;
            constexpr bool a_mn = KindTraits<KIND>::a_mn, b_mn = KindTraits<KIND>::b_mn;
            constexpr uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
            constexpr uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
            for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x)) {
                const Tile t = decode_tile_wide<KIND>(prm, st, tile, cursor);
                const bool two = t.a_boxes_peer > 0;
                if (!mbar_wait(smem_u32(&st->tmem_empty[0]), (use0 & 1u) ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc = make_idesc(a_mn, b_mn, t.n_mma);
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->full[stage]), phase, abort_flag, prm.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage_base + stage * kStageBytesW;
                    const uint64_t adesc0 = make_desc(a_addr, a_mn);
                    const uint64_t adesc1 = make_desc(a_addr + kARegion, a_mn);
                    const uint64_t bdesc = make_desc(a_addr + kARegionW, b_mn);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16(tmem_base, adesc0 + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step), idesc,
                                  (kb > 0 || ks > 0) ? 1u : 0u);
                    if (two) {
                        if (kb == 0) {
                            // the second accumulator may still be draining: the first half's MMAs above are already queued
                            if (!mbar_wait(smem_u32(&st->tmem_empty[1]), (use1 & 1u) ^ 1u, abort_flag, prm.status)) { ok = false; break; }
                            tc_fence_after();
                        }
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_bf16(tmem_base + kAccCols, adesc1 + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step),
                                      idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                    }
                    umma_commit(smem_u32(&st->empty[stage]));
                    if (++stage == kStagesW) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (t.nk > 0) umma_commit(smem_u32(&st->tmem_full[0]));
                else mbar_arrive(smem_u32(&st->tmem_full[0]));
                ++use0;
                if (two) ++use1;
            }
        }
    } else {
        // ===================== epilogue (warps 2..9) =====================
        const int quad = warp & 3;
        const int half = (warp - 2) >> 2;
        const int row = quad * 32 + lane;
        int cursor = 0, it = 0;
        bool ok = true;
        for (int rnd = 0, tile = dealt_tile<KIND>(0, blockIdx.x, gridDim.x); tile < total_tiles && ok;
                 tile = dealt_tile<KIND>(++rnd, blockIdx.x, gridDim.x), ++it) {
            const Tile t0 = decode_tile_wide<KIND>(prm, st, tile, cursor);
            if (!mbar_wait(smem_u32(&st->tmem_full[0]), (uint32_t)it & 1u, abort_flag, prm.status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16);
            const int chalf = t0.ncols >> 1;
            epilogue_row<KIND>(prm, t0, tacc, row, half * chalf, (half + 1) * chalf, st->epi_stage[warp - 2]);
            tc_fence_before();
            mbar_arrive(smem_u32(&st->tmem_empty[0]));
            if (t0.a_boxes_peer > 0) {
                const Tile t1 = second_half(t0);
                epilogue_row<KIND>(prm, t1, tacc + kAccCols, row, half * chalf, (half + 1) * chalf,
                                   st->epi_stage[warp - 2]);
                tc_fence_before();
                mbar_arrive(smem_u32(&st->tmem_empty[1]));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 row-major matrix [rows, cols] seen as a 2-D tensor, boxes of 64 columns x box_rows rows, 128-byte swizzle.
bool encode_2d(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows = 64)
{
    EncodeTiledFn fn = get_encode();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc_fill_maps(TcMaps &maps, const LayerMeta &m, const WsLayout &L, const WsPtrs &p, const modse_weights_t *w,
                  bool backward)
{
    const uint64_t panel_rows = L.hb / 64;
    bool ok = true;
    auto both = [&](CUtensorMap *m64, CUtensorMap *m128, const void *base, uint64_t rows, uint64_t cols) {
        ok = ok && encode_2d(m64, base, rows, cols, 64) && encode_2d(m128, base, rows, cols, 128);
    };
    both(&maps.xp, &maps.xp128, p.xp, L.Pmax, m.d);
    both(&maps.wgate, &maps.wgate128, w->w_gate, m.S, m.d);
    both(&maps.wup, &maps.wup128, w->w_up, m.S, m.d);
    both(&maps.wdown, &maps.wdown128, w->w_down, m.d, m.S);
    both(&maps.hm, &maps.hm128, p.hm, panel_rows, 64);
    if (backward) {
        both(&maps.dyp, &maps.dyp128, p.dyp, L.Pmax, m.d);
        both(&maps.da, &maps.da128, p.da, panel_rows, 64);
        both(&maps.db, &maps.db128, p.db, panel_rows, 64);
    } else {
        maps.dyp = maps.xp;   maps.dyp128 = maps.xp128;
        maps.da = maps.hm;    maps.da128 = maps.hm128;
        maps.db = maps.hm;    maps.db128 = maps.hm128;
    }
    return ok;
}

namespace {

TcParams make_params(const LayerMeta &m, const WsPtrs &p, const modse_wgrads_t *g, bool save, bool out_f32)
{
    TcParams prm{};
    prm.meta = m;
    prm.poffsets = p.poffsets;
    prm.ebase = p.ebase;
    prm.status = p.status;
    prm.pgate = p.pgate;
    prm.hm = (__nv_bfloat16 *)p.hm;
    prm.sp = (__nv_bfloat16 *)p.a_pre;
    prm.sq = (__nv_bfloat16 *)p.b_pre;
    prm.da = (__nv_bfloat16 *)p.da;
    prm.db = (__nv_bfloat16 *)p.db;
    prm.o = (float *)p.o;
    prm.dxp = (float *)p.dxp;
    if (g) {
        prm.dw_gate = (__nv_bfloat16 *)g->dw_gate;
        prm.dw_up = (__nv_bfloat16 *)g->dw_up;
        prm.dw_down = (__nv_bfloat16 *)g->dw_down;
    }
    prm.save = save ? 1 : 0;
    prm.out_f32 = out_f32 ? 1 : 0;
    return prm;
}

// Launches the two-CTA kernel with as many clusters as can be resident at once (tiles are dealt
// statically, so a cluster that is not resident would hold its share back).
template <int KIND>
cudaError_t launch_kind_pair(const TcMaps &maps, const TcParams &prm, int sms, cudaStream_t s, int *launches)
{
    auto kern = tc_grouped_gemm_pair<KIND>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes2);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(sms & ~1));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes2;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    static int max_clusters[6] = {0, 0, 0, 0, 0, 0};
    if (max_clusters[KIND] == 0) {
        int n = 0;
        e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
        if (e != cudaSuccess) return e;
        if (n < 1) return cudaErrorInvalidConfiguration;
        max_clusters[KIND] = n;
    }
    const int clusters = max_clusters[KIND] < sms / 2 ? max_clusters[KIND] : sms / 2;
    cfg.gridDim = dim3((unsigned)(2 * clusters));
    e = cudaLaunchKernelEx(&cfg, kern, maps, prm);
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

template <int KIND>
cudaError_t launch_kind_wide(const TcMaps &maps, const TcParams &prm, int grid, cudaStream_t s, int *launches)
{
    auto kern = tc_grouped_gemm_wide<KIND>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytesW);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytesW, s>>>(maps, prm);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

template <int KIND>
cudaError_t launch_kind(const TcMaps &maps, const TcParams &prm, int grid, int mask, cudaStream_t s, int *launches)
{
    if ((mask >> 8) & (1 << KIND)) return launch_kind_wide<KIND>(maps, prm, grid, s, launches);
    if (mask & (1 << KIND)) return launch_kind_pair<KIND>(maps, prm, grid, s, launches);
    auto kern = tc_grouped_gemm<KIND>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, kSmemBytes, s>>>(maps, prm);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

int sm_count(TcPlan &plan)
{
    if (plan.sm_count == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
            plan.sm_count = n;
        else
            plan.sm_count = 148;
    }
    return plan.sm_count;
}

}  // namespace

cudaError_t tc_launch(TcPlan &plan, TcKind kind, const TcMaps &maps, const LayerMeta &m, const WsPtrs &p,
                      const modse_wgrads_t *g, bool save, bool out_f32, cudaStream_t s, int *launches)
{
    const TcParams prm = make_params(m, p, g, save, out_f32);
    const int grid = sm_count(plan);
    const int mask = plan.tile_mask >= 0 ? plan.tile_mask : tc_pair_mask();
    switch (kind) {
    case TcUpGate: return launch_kind<TcUpGate>(maps, prm, grid, mask, s, launches);
    case TcDown: return launch_kind<TcDown>(maps, prm, grid, mask, s, launches);
    case TcDownDgrad: return launch_kind<TcDownDgrad>(maps, prm, grid, mask, s, launches);
    case TcDownWgrad: return launch_kind<TcDownWgrad>(maps, prm, grid, mask, s, launches);
    case TcUpGateDgrad: return launch_kind<TcUpGateDgrad>(maps, prm, grid, mask, s, launches);
    case TcUpGateWgrad: return launch_kind<TcUpGateWgrad>(maps, prm, grid, mask, s, launches);
    }
    return cudaErrorInvalidValue;
}

}  // namespace modse
