// Grouped GEMMs of the bf16 MoDSE layer on Blackwell tensor cores.
//
// Two persistent, warp-specialised kernel templates (one CTA per tile, or a pair
// of CTAs per tile) serve the six products of the layer (Sec. 3.1, Eq. 4 and its
// gradient); the accumulators (fp32) live in tensor memory (TMEM):
//
//   kind            product (per expert e, cp = padded rows, h = width)      K
//   UpGate          Hm = g * silu(xp Wg^T) * (xp Wu^T)      [cp, h]          d
//   Down            o  = Hm Wd_e^T                          [cp, d]  fp32    h
//   DownDgrad       dHm = g * (dyp Wd_e) -> dA, dB          [cp, h]          d
//   DownWgrad       dWd_e = dyp^T Hm                        [d, h]           cp
//   UpGateDgrad     dxp = dA Wg_e + dB Wu_e                 [cp, d]  fp32    2h
//   UpGateWgrad     dWg_e = dA^T xp, dWu_e = dB^T xp        [h, d]           cp
//
// Three tile shapes.  One CTA: 128 rows x up to 256 accumulator columns with two
// accumulators in flight (the epilogue of one tile overlaps the main loop of the
// next), or 256 rows (two 128-row halves that share the column operand, 2/3 of
// the shared-memory traffic per FLOP, but both accumulators belong to one tile).
// A pair of CTAs (cta_group::2, the default): 256 rows, each CTA stages its own
// 128 rows and half of the column operand and holds its half of the accumulator
// - the traffic of the second shape with the overlap of the first.
//
// Roles inside a CTA: warp 0 issues TMA loads into a ring of shared-memory
// stages (boxes of 64 elements x 64 or 128 rows, 128-byte swizzle), warp 1
// issues tcgen05.mma, warp 2 hands out tiles, warp 3 idles, and 8 or 16 epilogue
// warps (from warp 4 on) read the accumulator with tcgen05.ld - two or four warps
// per TMEM lane quadrant, each a run of the tile's columns - and run the fused
// epilogue.  A 256-row tile owns both accumulators, so its epilogue is exposed:
// there sixteen warps (four per scheduler) hide the latencies of the epilogue's
// loads, special-function chains and stores that eight cannot.
// Operands are consumed either K-major or MN-major
// straight from their row-major buffers (the instruction descriptor carries the
// major-ness), so the backward pass needs no transposed copies.
//
// (g = gate of the row's assignment: it is applied to the hidden row, in fp32,
// before the one rounding to bf16, so neither o nor dY needs a rounded gated
// copy; dyp is dY in group order, bit for bit.)
//
// For backward the up/gate epilogue saves, from its fp32 accumulators A and B,
// sp = B * silu'(A) and sq = silu(A) (bf16): then dA = dHm * sp, dB = dHm * sq, one
// rounded factor each instead of two rounded pre-activations.
//
// Activations that have the hidden axis as their width and feed an MMA (Hm, dA,
// dB) are stored as panels: for expert e, panel pc holds columns [64 pc,
// 64 pc + 64) of all cp rows contiguously, so that a single two-dimensional
// tensor map with 128-byte rows describes the whole buffer although the row
// length h differs from expert to expert.  sp and sq travel only from one
// epilogue to another, so they are stored the way an epilogue warp holds them:
// in blocks of 32 rows x 32 columns (2 KB), inside a block the 16-byte piece q
// of row r at byte q * 512 + r * 16.  A warp then writes and reads a block with
// four fully coalesced 512-byte accesses and no transposition.
//
// Tile order: experts by decreasing K, so the long tiles of wide experts (or of
// experts with many tokens) start first and the short ones fill the tail - the
// one-GPU form of the paper's expert-pair balancing (Sec. 3.2).  CTAs (or CTA
// pairs) take the next tile of that list from a counter in global memory (or,
// with the counter switched off, are dealt tiles round-robin).  Every output
// tile is computed by one CTA or one pair with its K blocks in ascending order
// either way, so the results do not depend on who ran which tile.  The counter is read by a
// warp of its own, which passes the tile indices to the three working roles
// through a small queue in shared memory: an atomic instruction inside the
// loop of the thread that issues the TMA loads cost the 128-row kernels a
// quarter of their speed (measured, even with the instruction never executed).
//
// Every wait is bounded; a wait that expires records kDevTimeout in the status
// word and the CTA drains and exits.
#include <cuda.h>

#include "tc_gemm.h"

namespace modse {

static int g_force_simt = 0;
static int g_default_plan = kTcDefaultPlan;
static int g_dynamic_tiles = 1;
static int g_wait_limit_ms = 2000;
static int g_skip_kind = -1, g_skip_tile = -1;
static int g_epi16_narrow = 0, g_epi16_wide = kTcDefaultEpi16Wide;   // bit per product: sixteen epilogue warps
static int g_epi16_pair = 0;

bool tc_force_simt() { return g_force_simt != 0; }
void tc_set_force_simt(int on) { g_force_simt = on ? 1 : 0; }
void tc_set_default_plan(int mask) { g_default_plan = mask & kTcPlanBits; }
int tc_default_plan() { return g_default_plan; }
void tc_set_dynamic_tiles(int on) { g_dynamic_tiles = on ? 1 : 0; }
void tc_set_wait_limit_ms(int ms) { g_wait_limit_ms = ms < 1 ? 1 : (ms > 60000 ? 60000 : ms); }
void tc_set_skip_tile(int kind, int tile) { g_skip_kind = kind; g_skip_tile = tile; }
void tc_set_epilogue_warps16(int narrow_mask, int wide_mask, int pair_mask)
{
    g_epi16_narrow = narrow_mask & 63;
    g_epi16_wide = wide_mask & 63;
    g_epi16_pair = pair_mask & 63;
}

namespace {

constexpr int kBoxBytes = 64 * 64 * 2;           // one TMA box: 64 rows of 128 bytes
constexpr int kARegion = 2 * kBoxBytes;          // 128 rows (or 128 MN elements) x 64 K
constexpr int kBRegion = 4 * kBoxBytes;          // up to 256 rows x 64 K
constexpr int kFirstEpiWarp = 4;                 // warps 0-2: TMA, MMA, tile hand-out; warp 3 idles (the epilogue starts on a warpgroup)
constexpr int kMaxEpiWarps = 16;
template <int EPI> constexpr int threads_of() { return 32 * (kFirstEpiWarp + EPI); }
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;
constexpr int kEpiRowBytes = 64;                 // a 32-element bf16 chunk of one row; 16-byte pieces XOR-swizzled
constexpr int kEpiBufBytes = 32 * kEpiRowBytes;  // one warp's 32 rows: 2 KB
template <int EPI> constexpr int epi_bytes() { return EPI * kEpiBufBytes; }   // one transposing buffer per epilogue warp
constexpr int kMaxStages = 6;
constexpr int kTileQ = 4;                        // tile indices in flight between the producer and the other roles

// 128-row tiles: 4 stages of 16 KB rows + 32 KB columns.  256-row tiles: 3 stages of 2 x 16 KB rows + 32 KB columns.
template <bool WIDE> struct Shape {
    static constexpr int kStages = WIDE ? 3 : 4;
    static constexpr int kRowRegion = WIDE ? 2 * kARegion : kARegion;
    static constexpr int kStageBytes = kRowRegion + kBRegion;
    static constexpr int kTileRows = WIDE ? 256 : 128;
};

struct TcParams {
    LayerMeta meta;
    const int *poffsets;
    const long long *ebase;
    int *status;
    int *tile_counter;            // this product's counter of tiles handed out (zero at launch)
    const float *pgate;           // gate of the assignment in each padded row (0 for padding)
    const int *ptoken_of;         // token of each padded row (-1 for padding)
    __nv_bfloat16 *hm, *da, *db;
    __nv_bfloat16 *sp, *sq;       // saved for backward: sp = B * silu'(A), sq = silu(A) (panel layout)
    float *o, *dxp;
    __nv_bfloat16 *dw_gate, *dw_up, *dw_down;
    float *dg_part;               // [slots][Pmax] partial row dots of the down dgrad with Hm
    float *scatter_out;           // fp32 [T, d] target of the scatter-adding epilogues
    unsigned long long wait_limit_ns;
    int Pmax, T;
    int save;
    int out_f32;   // weight gradients are written as fp32 instead of bf16
    int dynamic;   // tiles come from the global counter
    int skip_tile; // debugging: the producer that gets this tile stops without loading it (-1: none)
};

// control block behind the stages and the epilogue buffers
struct SmemTail {
    unsigned long long full[kMaxStages], empty[kMaxStages], tmem_full[2], tmem_empty[2], tq_full[kTileQ], tq_empty[kTileQ], tq_taken;
    unsigned int tmem_base;
    int abort_flag;
    int tile_q[kTileQ];
    int tstart[kMaxExperts + 1];
    unsigned short order[kMaxExperts];
};
template <bool WIDE, int EPI> constexpr size_t smem_bytes()
{
    return 1024 + (size_t)Shape<WIDE>::kStages * Shape<WIDE>::kStageBytes + epi_bytes<EPI>() + sizeof(SmemTail);
}
static_assert(smem_bytes<false, kMaxEpiWarps>() <= 232448 && smem_bytes<true, kMaxEpiWarps>() <= 232448,
              "shared memory per CTA");

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
// the same test with acquire semantics at cluster scope: what the partner CTA wrote before its (release.cluster)
// arrival is visible afterwards
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
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

// What a role needs to give up a wait: the CTA's abort flag, the status word and the time limit.
struct WaitCtx {
    volatile int *abort_flag;
    int *status;
    unsigned long long limit_ns;
};
// Bounded wait: false if the phase did not complete within the limit or the CTA is aborting.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    unsigned it = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++it & 255u) == 0) {
            if (*w.abort_flag || global_ns() - t0 > w.limit_ns) {
                *w.abort_flag = 1;
                atomicMax(w.status, kDevTimeout);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    unsigned it = 0;
    while (!mbar_try_wait_cluster(bar, parity)) {
        if ((++it & 255u) == 0) {
            if (*w.abort_flag || global_ns() - t0 > w.limit_ns) {
                *w.abort_flag = 1;
                atomicMax(w.status, kDevTimeout);
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
// Four rows y0..y3 of a tensor whose map has boxes one row high, into four consecutive 128-byte rows at dst
// (a row index outside the tensor reads zeros).
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y0, int y1,
                                            int y2, int y3)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3)
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

// The same copies inside a pair of CTAs (cta_group::2): the data lands in the issuing CTA's shared memory, the
// bytes are counted on a barrier of the pair's leader (`bar` is a shared::cluster address).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, uint32_t bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_rows_pair(uint32_t dst, const CUtensorMap *m64, const CUtensorMap *m128,
                                                   uint32_t bar, int x, int y, int nboxes)
{
    int i = 0;
    for (; i + 2 <= nboxes; i += 2) tma_load_2d_pair(dst + i * kBoxBytes, m128, bar, x, y + 64 * i);
    if (i < nboxes) tma_load_2d_pair(dst + i * kBoxBytes, m64, bar, x, y + 64 * i);
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

__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum)
        : "memory");
}
// arrives on the barrier at the same shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((unsigned short)3) : "memory");
}
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
// Arrival on a barrier of the partner CTA that also publishes what this thread wrote before it (release at
// cluster scope).  Slow - of the order of a microsecond - so only the tile hand-out uses it.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Arrival on a barrier of either CTA of the pair that publishes nothing: what it signals (a tile index read, an
// accumulator drained - ordered by the tcgen05 fence before it) is complete when the instruction issues.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
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

// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128 (one CTA) or 256 (a pair of CTAs).
__device__ __forceinline__ uint32_t make_idesc(bool a_mn, bool b_mn, int n, int m = 128)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Static hand-out (the global counter switched off): tiles are dealt to the CTAs in rounds of one tile each.
// The tile list is sorted by decreasing length of the K loop, so within a round the first CTA gets the
// longest tile; where K is the expert's width (down, up/gate dgrad) dealing every round in the same
// direction hands the same CTAs the longer tile of every round (12 % above the mean load for the
// benchmark's widths), so odd rounds run through the CTAs in reverse order, which evens that out (5.5 %).
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
    int a_boxes_peer;                 // 256-row tiles: boxes of the second 128-row half
};

// tiles (rows, columns) and K blocks of one expert
template <int KIND, bool WIDE>
__device__ __forceinline__ void expert_shape(int cp, int h, int d, int &mt, int &nt, int &nk)
{
    constexpr int R = WIDE ? 256 : 128;
    if constexpr (KIND == TcUpGate)      { mt = (cp + R - 1) / R; nt = (h + 127) / 128; nk = d / 64; }
    if constexpr (KIND == TcDown)        { mt = (cp + R - 1) / R; nt = (d + 255) / 256; nk = h / 64; }
    if constexpr (KIND == TcDownDgrad)   { mt = (cp + R - 1) / R; nt = (h + 255) / 256; nk = d / 64; }
    if constexpr (KIND == TcDownWgrad)   { mt = (d + R - 1) / R;  nt = (h + 255) / 256; nk = cp / 64; }
    if constexpr (KIND == TcUpGateDgrad) { mt = (cp + R - 1) / R; nt = (d + 255) / 256; nk = 2 * (h / 64); }
    if constexpr (KIND == TcUpGateWgrad) { mt = 2 * ((h + R - 1) / R); nt = (d + 255) / 256; nk = cp / 64; }
}

// Tile `tile` of the sorted list.  128-row tiles: the tile itself.  256-row tiles: its first half (rows
// m0 .. m0+127); a_boxes_peer carries the second half's boxes.
template <int KIND, bool WIDE>
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
    expert_shape<KIND, WIDE>(t.cp, t.h, d, mt, nt, nk);
    const int local = tile - st->tstart[cursor];
    // Order of an expert's tiles (the ~148 tiles in flight should share operands through L2):
    // row-block fastest where the column operand is the big one (weights of the up/gate GEMM, Hm
    // panels of the down wgrad), column-block fastest where all column blocks of one row block
    // fit in flight at once (d / 256 = 8 column blocks), so the row operand is read once.
    constexpr bool n_fastest = (KIND == TcDown || KIND == TcUpGateDgrad || KIND == TcUpGateWgrad);
    int mb, nb;
    tile_coords<n_fastest>(local, mt, nt, group_row_tiles(d, Shape<WIDE>::kTileRows), mb, nb);
    t.nk = nk;
    t.which = 0;
    int row_extent;                       // extent of the tile's row dimension for this expert
    if constexpr (KIND == TcDownWgrad) row_extent = d;
    else if constexpr (KIND == TcUpGateWgrad) { row_extent = t.h; t.which = mb & 1; mb >>= 1; }
    else row_extent = t.cp;
    t.m0 = mb * Shape<WIDE>::kTileRows;
    t.mrows = max(0, min(128, row_extent - t.m0));
    t.a_boxes = t.mrows / 64;
    t.a_boxes_peer = WIDE ? max(0, min(128, row_extent - t.m0 - 128)) / 64 : 0;
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

// Row-operand boxes of one 128-row half of k-block kb.
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

// Column-operand boxes of k-block kb of a tile.
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

// ---------------------------------------------------------------------------
// Epilogue helpers.  A warp's 32 threads each hold 32 values of their own row.
// ---------------------------------------------------------------------------
// Byte offset of 16-byte piece q of row r in a warp's 2 KB buffer.  Rows are 64 bytes; the piece index is
// XORed with (r / 2) % 4, so that both access patterns are free of bank conflicts: eight lanes writing the
// same piece of eight consecutive rows, and eight lanes reading all pieces of two consecutive rows.
__device__ __forceinline__ int epi_piece(int r, int q) { return r * kEpiRowBytes + ((q ^ ((r >> 1) & 3)) << 4); }

__device__ __forceinline__ void pack_bf16x32(const float (&v)[32], uint4 (&w4)[4])
{
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
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&t);
}

// Row-by-row stores of a warp's chunk would touch 32 lines with 16 bytes each per instruction, so the chunk is
// transposed through shared memory: afterwards four neighbouring lanes cover the 64 bytes of one row and an
// instruction moves eight whole 64-byte row segments.  `own` points at this thread's own row chunk.
// rows_valid: rows of this warp (0..32, counted from the warp's first row) that may be written.
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
    pack_bf16x32(v, w4);
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

__device__ __forceinline__ void red_add_f32x4(float *addr, const uint4 &v)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
                 ::"l"(addr), "f"(__uint_as_float(v.x)), "f"(__uint_as_float(v.y)), "f"(__uint_as_float(v.z)),
                   "f"(__uint_as_float(v.w))
                 : "memory");
}

// The warp's 32 rows x 32 fp32 values are added into rows tok (one per lane; -1: no row) of a [T, row_stride]
// fp32 matrix at column col0: the same transposition, then 16-byte reductions.  With at most two rows added
// into a zeroed element the result does not depend on their order (0 + a + b == 0 + b + a).
__device__ __forceinline__ void red_f32x32_staged(unsigned char *stg, int lane, float *base, long long row_stride, int tok,
                                                  int col0, const float (&v)[32])
{
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4 *>(stg + epi_piece(lane, q)) =
                make_uint4(__float_as_uint(v[hh * 16 + 4 * q]), __float_as_uint(v[hh * 16 + 4 * q + 1]),
                           __float_as_uint(v[hh * 16 + 4 * q + 2]), __float_as_uint(v[hh * 16 + 4 * q + 3]));
        __syncwarp();
        const int q = lane & 3;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int rr = 8 * j + (lane >> 2);
            const int tk = __shfl_sync(0xFFFFFFFFu, tok, rr);
            const uint4 val = *reinterpret_cast<const uint4 *>(stg + epi_piece(rr, q));
            if (tk >= 0) red_add_f32x4(base + (long long)tk * row_stride + col0 + hh * 16 + q * 4, val);
        }
        __syncwarp();
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

// The tile's 32-column chunks are split into NQ contiguous runs, one per warp of the lane quadrant.
template <int NQ>
__device__ __forceinline__ void chunk_range(int ncols, int cq, int &c_begin, int &c_end)
{
    const int per = ((ncols >> 5) + NQ - 1) / NQ;
    c_begin = min(ncols, cq * per * 32);
    c_end = min(ncols, c_begin + per * 32);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// Epilogue of one 128-row (half) tile for one thread: accumulator row `row`, run cq of the tile's 32-column
// chunks (NQ = epilogue warps per TMEM lane quadrant).
//   VAR = 1 selects the product's fused variant: DownDgrad also writes the partial row dot of its
//   accumulator with Hm (for dg); Down and UpGateDgrad add their rows into fp32 [T, d] token rows.
template <int KIND, int VAR, int NQ>
__device__ __forceinline__ void epilogue_row(const TcParams &prm, const Tile &t, uint32_t tacc, int row, int lane, int cq,
                                             unsigned char *stg)
{
    const int d = prm.meta.d, S = prm.meta.S;
    const bool have_acc = t.nk > 0;
    int c_first, c_end;
    chunk_range<NQ>(t.ncols, cq, c_first, c_end);
    constexpr int c_step = 32;
    auto panel_index = [&](int c) {
        const int col = t.n0 + c;
        return ((size_t)(t.pbase + (col >> 6) * t.cp + t.m0 + row) << 6) + (col & 63);
    };
    // first element of the 32 x 32 block of sp / sq that holds this warp's rows and columns t.n0 + c ..
    auto block_index = [&](int c) {
        return ((size_t)t.pbase << 6) + ((size_t)((t.n0 + c) >> 5) * (size_t)(t.cp >> 5) + (size_t)((t.m0 + row) >> 5)) * 1024;
    };
    if constexpr (KIND == TcUpGate) {
        // 32-column chunks in two halves of 16 accumulator columns (registers: sixteen epilogue warps leave 96
        // per thread); the chunk's gated hidden values are kept packed and leave as 64-byte row segments
        const float gate = prm.pgate[t.prow0 + t.m0 + row];
        for (int c = c_first; c < c_end; c += c_step) {
            uint4 hw4[4];
            uint4 *dp = nullptr, *dq = nullptr;
            if (prm.save) {
                const size_t blk = block_index(c);
                dp = reinterpret_cast<uint4 *>(prm.sp + blk) + lane;
                dq = reinterpret_cast<uint4 *>(prm.sq + blk) + lane;
            }
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2) {
                uint32_t ra[16], rb[16];
                tmem_ld16(tacc + c + 16 * s2, ra);
                tmem_ld16(tacc + t.ncols + c + 16 * s2, rb);
                tmem_ld_wait();
                uint32_t wh[8];
                if (prm.save) {
                    uint32_t wp[8], wq[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float sq2[2], sp2[2], hm2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const float av = __uint_as_float(ra[2 * i + u]), bv = __uint_as_float(rb[2 * i + u]);
                            const float sg = __fdividef(1.0f, 1.0f + __expf(-av));   // ex2 + rcp: a full-precision division here slows the MMA warp
                            sq2[u] = av * sg;
                            sp2[u] = bv * sg * (1.0f + av * (1.0f - sg));
                            hm2[u] = gate * (sq2[u] * bv);
                        }
                        wp[i] = pack_bf16x2(sp2[0], sp2[1]);
                        wq[i] = pack_bf16x2(sq2[0], sq2[1]);
                        wh[i] = pack_bf16x2(hm2[0], hm2[1]);
                    }
                    dp[(2 * s2) * 32] = make_uint4(wp[0], wp[1], wp[2], wp[3]);
                    dp[(2 * s2 + 1) * 32] = make_uint4(wp[4], wp[5], wp[6], wp[7]);
                    dq[(2 * s2) * 32] = make_uint4(wq[0], wq[1], wq[2], wq[3]);
                    dq[(2 * s2 + 1) * 32] = make_uint4(wq[4], wq[5], wq[6], wq[7]);
                } else {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float hm2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const float av = __uint_as_float(ra[2 * i + u]), bv = __uint_as_float(rb[2 * i + u]);
                            hm2[u] = gate * (av * __fdividef(1.0f, 1.0f + __expf(-av)) * bv);
                        }
                        wh[i] = pack_bf16x2(hm2[0], hm2[1]);
                    }
                }
                hw4[2 * s2] = make_uint4(wh[0], wh[1], wh[2], wh[3]);
                hw4[2 * s2 + 1] = make_uint4(wh[4], wh[5], wh[6], wh[7]);
            }
            store_u4x4_staged(stg, lane, reinterpret_cast<unsigned char *>(prm.hm + panel_index(c)), 128, hw4, 32);
        }
    } else if constexpr (KIND == TcDown || KIND == TcUpGateDgrad) {
        if constexpr (VAR == 1) {
            int tok = prm.ptoken_of[t.prow0 + t.m0 + row];
            if (tok >= prm.T) {                      // not a token of this batch: recorded, row skipped
                atomicMax(prm.status, kDevBounds);
                tok = -1;
            }
            for (int c = c_first; c < c_end; c += c_step) {
                uint32_t r[32];
                float v[32];
                tmem_ld32(tacc + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                red_f32x32_staged(stg, lane, prm.scatter_out, d, tok, t.n0 + c, v);
            }
        } else {
            float *out = (KIND == TcDown ? prm.o : prm.dxp) + (size_t)(t.prow0 + t.m0 + row) * d + t.n0;
            for (int c = c_first; c < c_end; c += c_step) {
                uint32_t r[32];
                float v[32];
                tmem_ld32(tacc + c, r);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
                store_f32x32_staged(stg, lane, out + c, d, v);
            }
        }
    } else if constexpr (KIND == TcDownDgrad) {
        // dA = dHm * sp, dB = dHm * sq with dHm = gate * acc, 32-column chunks in two halves of 16 columns;
        // the saved factors (and, for the row dot, Hm) of a chunk are requested before its accumulator
        const float gate = prm.pgate[t.prow0 + t.m0 + row];
        float rowdot = 0.f;                // VAR 1: sum over this thread's columns of acc * Hm
        for (int c = c_first; c < c_end; c += c_step) {
            const uint4 *psrc = reinterpret_cast<const uint4 *>(prm.sp + block_index(c)) + lane;
            const uint4 *qsrc = reinterpret_cast<const uint4 *>(prm.sq + block_index(c)) + lane;
            uint4 pown[4], qown[4];        // this thread's row of the saved factors (block layout: no transposition)
#pragma unroll
            for (int q = 0; q < 4; ++q) { pown[q] = psrc[q * 32]; qown[q] = qsrc[q * 32]; }
            uint4 hown[4];
            if constexpr (VAR == 1) {
                uint4 hraw[4];             // Hm, transposed: entry j belongs to row 8j + lane/4 of this warp
                load_bf16x32_transposed(prm.hm + panel_index(c), 64, lane, hraw);
                untranspose_rows(stg, lane, hraw, hown);
            }
            uint4 da4[4], db4[4];
#pragma unroll
            for (int s2 = 0; s2 < 2; ++s2) {
                uint32_t r[16];
                tmem_ld16(tacc + c + 16 * s2, r);
                tmem_ld_wait();
                uint32_t wa[8], wb[8];
#pragma unroll
                for (int q4 = 0; q4 < 2; ++q4) {
                    const uint4 p4 = pown[2 * s2 + q4], q4v = qown[2 * s2 + q4];
                    const uint32_t pw[4] = {p4.x, p4.y, p4.z, p4.w};
                    const uint32_t qw[4] = {q4v.x, q4v.y, q4v.z, q4v.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int e0 = q4 * 8 + 2 * i;
                        const float a0 = __uint_as_float(r[e0]), a1 = __uint_as_float(r[e0 + 1]);
                        if constexpr (VAR == 1) {
                            const uint4 h4 = hown[2 * s2 + q4];
                            const uint32_t hw[4] = {h4.x, h4.y, h4.z, h4.w};
                            rowdot = fmaf(a0, bf16_lo(hw[i]), rowdot);
                            rowdot = fmaf(a1, bf16_hi(hw[i]), rowdot);
                        }
                        const float dh0 = gate * a0, dh1 = gate * a1;
                        wa[q4 * 4 + i] = pack_bf16x2(dh0 * bf16_lo(pw[i]), dh1 * bf16_hi(pw[i]));
                        wb[q4 * 4 + i] = pack_bf16x2(dh0 * bf16_lo(qw[i]), dh1 * bf16_hi(qw[i]));
                    }
                }
                da4[2 * s2] = make_uint4(wa[0], wa[1], wa[2], wa[3]);
                da4[2 * s2 + 1] = make_uint4(wa[4], wa[5], wa[6], wa[7]);
                db4[2 * s2] = make_uint4(wb[0], wb[1], wb[2], wb[3]);
                db4[2 * s2 + 1] = make_uint4(wb[4], wb[5], wb[6], wb[7]);
            }
            const size_t idx = panel_index(c);
            store_u4x4_staged(stg, lane, reinterpret_cast<unsigned char *>(prm.da + idx), 128, da4, 32);
            store_u4x4_staged(stg, lane, reinterpret_cast<unsigned char *>(prm.db + idx), 128, db4, 32);
        }
        // one partial per (row, 256-column tile, run of the columns); a warp without a chunk writes its zero
        if constexpr (VAR == 1)
            prm.dg_part[(size_t)((t.n0 >> 8) * NQ + cq) * prm.Pmax + t.prow0 + t.m0 + row] = rowdot;
    } else if constexpr (KIND == TcDownWgrad) {
        const size_t oidx = (size_t)(t.m0 + row) * S + t.ho + t.n0;
        for (int c = c_first; c < c_end; c += c_step) {
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
            const int rows_valid = t.mrows - (row - lane);
            if (prm.out_f32) store_f32x32_staged(stg, lane, reinterpret_cast<float *>(prm.dw_down) + oidx + c, S, v, rows_valid);
            else store_bf16x32_staged(stg, lane, prm.dw_down + oidx + c, S, v, rows_valid);
        }
    } else {
        __nv_bfloat16 *obase = t.which ? prm.dw_up : prm.dw_gate;
        const size_t oidx = (size_t)(t.ho + t.m0 + row) * d + t.n0;
        for (int c = c_first; c < c_end; c += c_step) {
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

// ---------------------------------------------------------------------------
// Schedule: experts by decreasing K, tiles of an expert contiguous.  `key` and
// `ntile` are scratch arrays of kMaxExperts ints (the epilogue buffers serve).
// ---------------------------------------------------------------------------
template <int KIND, bool WIDE>
__device__ __forceinline__ void build_schedule(const TcParams &prm, SmemTail *st, int *key, int *ntile, int tid)
{
    const int N = prm.meta.N, d = prm.meta.d;
    for (int e = tid; e < N; e += (int)blockDim.x) {
        const int cp = prm.poffsets[e + 1] - prm.poffsets[e];
        const int h = prm.meta.hoff[e + 1] - prm.meta.hoff[e];
        int mt, nt, nk;
        expert_shape<KIND, WIDE>(cp, h, d, mt, nt, nk);
        // a group outside the padded row space (or not padded to whole tiles) is recorded and gets no tiles
        const bool sane = prm.poffsets[e] >= 0 && cp >= 0 && prm.poffsets[e + 1] <= prm.Pmax && (prm.poffsets[e] & 127) == 0 &&
                          (cp & 127) == 0;
        if (!sane && blockIdx.x == 0) atomicMax(prm.status, kDevBounds);
        ntile[e] = sane ? mt * nt : 0;
        key[e] = nk;
    }
    __syncthreads();
    for (int e = tid; e < N; e += (int)blockDim.x) {
        int rank = 0;
        const int ke = key[e];
        for (int f = 0; f < N; ++f) {
            const int kf = key[f];
            rank += (kf > ke) || (kf == ke && f < e);
        }
        st->order[rank] = (unsigned short)e;
    }
    __syncthreads();
    if (tid == 0) {
        int acc = 0;
        for (int i = 0; i < N; ++i) { st->tstart[i] = acc; acc += ntile[st->order[i]]; }
        st->tstart[N] = acc;
    }
}

// The tile warp's loop: takes tile after tile from the global counter and hands each to the three working roles
// through the queue; ends with -1 when the list is exhausted.  It stays one tile ahead of the TMA leader, the
// most advanced role (tq_taken): enough to hide the counter's round trip, and no more, because a tile taken
// early is a tile another CTA cannot take.
__device__ __forceinline__ void hand_out_tiles(const TcParams &prm, SmemTail *st, int total, const WaitCtx &w)
{
    for (int it = 0;; ++it) {
        const int slot = it & (kTileQ - 1);
        const uint32_t ph = (uint32_t)(it / kTileQ) & 1u;
        if (it > 0 && !mbar_wait(smem_u32(&st->tq_taken), (uint32_t)(it - 1) & 1u, w)) return;   // the leader has started on tile it - 1
        if (!mbar_wait(smem_u32(&st->tq_empty[slot]), ph ^ 1u, w)) return;
        int tile = atomicAdd(prm.tile_counter, 1);
        if (tile >= total) tile = -1;
        st->tile_q[slot] = tile;
        mbar_arrive(smem_u32(&st->tq_full[slot]));
        if (tile < 0) return;
    }
}

// Consumer side: the it-th tile of this CTA (-1: no more), not yet released.
template <int KIND>
__device__ __forceinline__ int peek_tile(const TcParams &prm, SmemTail *st, int it, int total, const WaitCtx &w, bool &ok)
{
    if (!prm.dynamic) {
        const int tile = dealt_tile<KIND>(it, blockIdx.x, gridDim.x);
        return tile >= total ? -1 : tile;
    }
    const int slot = it & (kTileQ - 1);
    const uint32_t ph = (uint32_t)(it / kTileQ) & 1u;
    if (!mbar_wait(smem_u32(&st->tq_full[slot]), ph, w)) { ok = false; return -1; }
    return *reinterpret_cast<volatile int *>(&st->tile_q[slot]);
}
__device__ __forceinline__ void release_tile(const TcParams &prm, SmemTail *st, int it)
{
    if (prm.dynamic) mbar_arrive(smem_u32(&st->tq_empty[it & (kTileQ - 1)]));
}

// ---------------------------------------------------------------------------
// The kernel.  WIDE: 256-row tiles (two halves sharing the column operand; both
// accumulators belong to the tile).  VAR 1: the product's fused variant -
// UpGate gathers its rows from x by token index (every lane of the producer
// warp issues one four-row gather per half and k-block), DownDgrad writes row
// dots for dg, Down / UpGateDgrad add into token rows.
// ---------------------------------------------------------------------------
template <int KIND, bool WIDE, int VAR, int EPI>
__global__ void __launch_bounds__(threads_of<EPI>(), 1)
tc_grouped_gemm(const __grid_constant__ TcMaps maps, const __grid_constant__ TcParams prm)
{
    constexpr int NQ = EPI / 4;                  // epilogue warps per TMEM lane quadrant
    using Sh = Shape<WIDE>;
    constexpr int kStages = Sh::kStages;
    constexpr int kStageBytes = Sh::kStageBytes;
    constexpr bool kGather = (KIND == TcUpGate && VAR == 1);
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    unsigned char *smem = smem_raw + pad;
    const uint32_t stage_base = raw + pad;
    unsigned char *epi_bufs = smem + (size_t)kStages * kStageBytes;
    SmemTail *st = reinterpret_cast<SmemTail *>(epi_bufs + EPI * kEpiBufBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&st->full[s]), 1);
            mbar_init(smem_u32(&st->empty[s]), 1);
        }
        mbar_init(smem_u32(&st->tmem_full[0]), 1);
        mbar_init(smem_u32(&st->tmem_full[1]), 1);
        mbar_init(smem_u32(&st->tmem_empty[0]), 32 * EPI);
        mbar_init(smem_u32(&st->tmem_empty[1]), 32 * EPI);
        mbar_init(smem_u32(&st->tq_taken), 1);
        for (int s = 0; s < kTileQ; ++s) {
            mbar_init(smem_u32(&st->tq_full[s]), 1);
            mbar_init(smem_u32(&st->tq_empty[s]), 2 + EPI);   // the TMA leader, the MMA thread and one lane of each epilogue warp
        }
        st->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    build_schedule<KIND, WIDE>(prm, st, reinterpret_cast<int *>(epi_bufs), reinterpret_cast<int *>(epi_bufs) + kMaxExperts, tid);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&st->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = st->tmem_base;
    const int total_tiles = st->tstart[prm.meta.N];
    const WaitCtx wc{&st->abort_flag, prm.status, prm.wait_limit_ns};

    if (warp == 0) {
        // ===================== TMA producer =====================
        if (kGather || lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                int tile = -1;
                if (lane == 0) {
                    tile = peek_tile<KIND>(prm, st, it, total_tiles, wc, ok);
                    if (ok) {
                        release_tile(prm, st, it);
                        if (prm.dynamic) mbar_arrive(smem_u32(&st->tq_taken));
                    }
                }
                if constexpr (kGather) {
                    tile = __shfl_sync(0xFFFFFFFFu, tile, 0);
                    ok = __shfl_sync(0xFFFFFFFFu, (int)ok, 0) != 0;
                }
                if (!ok || tile < 0 || tile == prm.skip_tile) break;
                const Tile t0 = decode_tile<KIND, WIDE>(prm, st, tile, cursor);
                const Tile t1 = second_half(t0);
                const uint32_t bytes = (uint32_t)(t0.a_boxes + (WIDE ? t1.a_boxes : 0) + t0.b_boxes) * kBoxBytes;
                int4 tok0 = make_int4(-1, -1, -1, -1), tok1 = make_int4(-1, -1, -1, -1);
                if constexpr (kGather) {
                    // rows 4 lane .. 4 lane + 3 of each half: their tokens (pad rows and rows past the group: -1)
                    const int r0 = t0.prow0 + t0.m0 + 4 * lane;
                    if (4 * lane < t0.mrows) tok0 = *reinterpret_cast<const int4 *>(prm.ptoken_of + r0);
                    if (WIDE && 4 * lane < t1.mrows) tok1 = *reinterpret_cast<const int4 *>(prm.ptoken_of + r0 + 128);
                }
                for (int kb = 0; kb < t0.nk; ++kb) {
                    // the leader waits for the stage; with all lanes at work they take its verdict, so that none
                    // leaves the loop alone
                    bool got = (lane == 0) ? mbar_wait(smem_u32(&st->empty[stage]), phase ^ 1u, wc) : true;
                    if constexpr (kGather) got = __shfl_sync(0xFFFFFFFFu, (int)got, 0) != 0;
                    if (!got) { ok = false; break; }
                    const uint32_t bar = smem_u32(&st->full[stage]);
                    const uint32_t a_dst = stage_base + stage * kStageBytes;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar, bytes);
                        if constexpr (!kGather) {
                            load_rows<KIND>(maps, t0, kb, a_dst, bar);
                            if constexpr (WIDE) load_rows<KIND>(maps, t1, kb, a_dst + kARegion, bar);
                        }
                        load_cols<KIND>(maps, t0, kb, a_dst + Sh::kRowRegion, bar);
                    }
                    if constexpr (kGather) {
                        __syncwarp();                         // the byte count is posted before any copy can complete
                        if (4 * lane < 64 * t0.a_boxes)
                            tma_gather4(a_dst + lane * 512, &maps.xg, bar, kb * 64, tok0.x, tok0.y, tok0.z, tok0.w);
                        if (WIDE && 4 * lane < 64 * t1.a_boxes)
                            tma_gather4(a_dst + kARegion + lane * 512, &maps.xg, bar, kb * 64, tok1.x, tok1.y, tok1.z, tok1.w);
                    }
                    ++issued;
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok && lane == 0) {
                // let the copies already issued land before the CTA leaves: wait (bounded) for
                // the current phase of every stage that has had a load
                const int n = issued < kStages ? (int)issued : kStages;
                for (int i = 1; i <= n; ++i) {
                    int s = stage - i;
                    uint32_t ph = phase;
                    if (s < 0) { s += kStages; ph ^= 1u; }
                    const unsigned long long tb = global_ns();
                    while (!mbar_try_wait(smem_u32(&st->full[s]), ph) && global_ns() - tb < prm.wait_limit_ns) {}
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            uint32_t use0 = 0, use1 = 0;         // WIDE: how often each accumulator has been handed to the epilogue
            bool ok = true;
            constexpr bool a_mn = KindTraits<KIND>::a_mn, b_mn = KindTraits<KIND>::b_mn;
            constexpr uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
            constexpr uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
            for (int it = 0; ok; ++it) {
                const int tile = peek_tile<KIND>(prm, st, it, total_tiles, wc, ok);
                if (!ok) break;
                release_tile(prm, st, it);
                if (tile < 0) break;
                const Tile t = decode_tile<KIND, WIDE>(prm, st, tile, cursor);
                const uint32_t idesc = make_idesc(a_mn, b_mn, t.n_mma);
                if constexpr (!WIDE) {
                    const int acc = it & 1;
                    const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                    if (!mbar_wait(smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, wc)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t tacc = tmem_base + (uint32_t)(acc * kAccCols);
                    for (int kb = 0; kb < t.nk; ++kb) {
                        if (!mbar_wait(smem_u32(&st->full[stage]), phase, wc)) { ok = false; break; }
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
                } else {
                    const bool two = t.a_boxes_peer > 0;
                    if (!mbar_wait(smem_u32(&st->tmem_empty[0]), (use0 & 1u) ^ 1u, wc)) { ok = false; break; }
                    tc_fence_after();
                    for (int kb = 0; kb < t.nk; ++kb) {
                        if (!mbar_wait(smem_u32(&st->full[stage]), phase, wc)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t a_addr = stage_base + stage * kStageBytes;
                        const uint64_t adesc0 = make_desc(a_addr, a_mn);
                        const uint64_t adesc1 = make_desc(a_addr + kARegion, a_mn);
                        const uint64_t bdesc = make_desc(a_addr + Sh::kRowRegion, b_mn);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_bf16(tmem_base, adesc0 + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step), idesc,
                                      (kb > 0 || ks > 0) ? 1u : 0u);
                        if (two) {
                            if (kb == 0) {
                                // the second accumulator may still be draining: the first half's MMAs above are already queued
                                if (!mbar_wait(smem_u32(&st->tmem_empty[1]), (use1 & 1u) ^ 1u, wc)) { ok = false; break; }
                                tc_fence_after();
                            }
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                umma_bf16(tmem_base + kAccCols, adesc1 + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step),
                                          idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                        }
                        umma_commit(smem_u32(&st->empty[stage]));
                        if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    if (t.nk > 0) umma_commit(smem_u32(&st->tmem_full[0]));
                    else mbar_arrive(smem_u32(&st->tmem_full[0]));
                    ++use0;
                    if (two) ++use1;
                }
            }
        }
    } else if (warp == 2) {
        // ===================== tile hand-out =====================
        if (lane == 0 && prm.dynamic) hand_out_tiles(prm, st, total_tiles, wc);
    } else if (warp >= kFirstEpiWarp) {
        // ===================== epilogue =====================
        const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
        const int cq = (warp - kFirstEpiWarp) >> 2;   // which of the quadrant's NQ warps: which run of the tile's columns
        const int row = quad * 32 + lane;
        unsigned char *stg = epi_bufs + (warp - kFirstEpiWarp) * kEpiBufBytes;
        int cursor = 0;
        bool ok = true;
        for (int it = 0; ok; ++it) {
            const int tile = peek_tile<KIND>(prm, st, it, total_tiles, wc, ok);
            if (!ok) break;
            __syncwarp();
            if (lane == 0) release_tile(prm, st, it);
            if (tile < 0) break;
            const Tile t = decode_tile<KIND, WIDE>(prm, st, tile, cursor);
            if constexpr (!WIDE) {
                const int acc = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&st->tmem_full[acc]), acc_phase, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccCols);
                epilogue_row<KIND, VAR, NQ>(prm, t, tacc, row, lane, cq, stg);
                tc_fence_before();
                mbar_arrive(smem_u32(&st->tmem_empty[acc]));
            } else {
                if (!mbar_wait(smem_u32(&st->tmem_full[0]), (uint32_t)it & 1u, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16);
                epilogue_row<KIND, VAR, NQ>(prm, t, tacc, row, lane, cq, stg);
                tc_fence_before();
                mbar_arrive(smem_u32(&st->tmem_empty[0]));
                if (t.a_boxes_peer > 0) {
                    const Tile t1 = second_half(t);
                    epilogue_row<KIND, VAR, NQ>(prm, t1, tacc + kAccCols, row, lane, cq, stg);
                    tc_fence_before();
                    mbar_arrive(smem_u32(&st->tmem_empty[1]));
                }
            }
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

// ---------------------------------------------------------------------------
// Two-CTA kernel (cta_group::2).  A cluster of two CTAs on neighbouring SMs
// computes one 256-row tile with M = 256 instructions: each CTA stages its own
// 128 rows of the row operand and HALF of the column operand (32 KB per k-block
// instead of the 48 KB of the 128-row kernel, for the same MMA work per CTA), the
// tensor cores of both SMs read both halves, and each CTA's tensor memory holds
// the accumulator rows of its own half - 256 columns per tile, so two tiles fit
// and the epilogue of one overlaps the main loop of the next, which a single CTA
// cannot do for a 256-row tile.  The leader (cluster rank 0) issues the MMAs.
//   full[s]        leader only: its producer posts the bytes of both CTAs, the
//                  copies of both complete on it
//   empty[s]       one per CTA; tcgen05.commit arrives on both
//   tmem_full[a]   one per CTA; tcgen05.commit arrives on both
//   tmem_empty[a]  leader only; one arrival per epilogue warp of both CTAs
// Tiles come from the global counter through the leader's tile warp (or are dealt to the clusters round-robin).
// ---------------------------------------------------------------------------
constexpr int kPairStages = 6;
constexpr int kPairHalfB = 2 * kBoxBytes;                     // this CTA's half of the column operand: up to 128 x 64
constexpr int kPairStageBytes = kARegion + kPairHalfB;        // 32 KB
template <int EPI> constexpr size_t pair_smem_bytes()
{
    return 1024 + (size_t)kPairStages * kPairStageBytes + epi_bytes<EPI>() + sizeof(SmemTail);
}
static_assert(pair_smem_bytes<kMaxEpiWarps>() <= 232448, "shared memory per CTA");
static_assert(kPairStages <= kMaxStages, "barrier arrays");

// Accumulator columns of a pair tile (each CTA stages half of them): a multiple of 128, so that a half is whole
// 64-column boxes; columns past the tile's own are computed from whatever lies beside them and never stored.
template <int KIND>
__device__ __forceinline__ int pair_n_mma(const Tile &t)
{
    if constexpr (KIND == TcUpGate) return 2 * t.ncols;       // gate columns in the leader, up columns in its partner
    else return (t.ncols + 127) & ~127;
}

// This CTA's half of the column operand of k-block kb.
template <int KIND>
__device__ __forceinline__ void load_cols_pair(const TcMaps &maps, const Tile &t, int rank, int kb, uint32_t dst, uint32_t bar)
{
    const int half = pair_n_mma<KIND>(t) / 2, nb = half / 64;
    if constexpr (KIND == TcUpGate) {
        if (rank == 0) tma_load_rows_pair(dst, &maps.wgate, &maps.wgate128, bar, kb * 64, t.ho + t.n0, nb);
        else tma_load_rows_pair(dst, &maps.wup, &maps.wup128, bar, kb * 64, t.ho + t.n0, nb);
    } else if constexpr (KIND == TcDown) {
        tma_load_rows_pair(dst, &maps.wdown, &maps.wdown128, bar, t.ho + kb * 64, t.n0 + rank * half, nb);
    } else if constexpr (KIND == TcDownDgrad) {
        for (int i = 0; i < nb; ++i)
            tma_load_2d_pair(dst + i * kBoxBytes, &maps.wdown, bar, t.ho + t.n0 + rank * half + 64 * i, kb * 64);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < nb; ++i)
            tma_load_2d_pair(dst + i * kBoxBytes, &maps.hm, bar, 0, t.pbase + ((t.n0 + rank * half) / 64 + i) * t.cp + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int hk = t.h / 64;
        const bool second = kb >= hk;
        const int kk = second ? kb - hk : kb;
        const CUtensorMap *bm = second ? &maps.wup : &maps.wgate;
        for (int i = 0; i < nb; ++i) tma_load_2d_pair(dst + i * kBoxBytes, bm, bar, t.n0 + rank * half + 64 * i, t.ho + kk * 64);
    } else {
        for (int i = 0; i < nb; ++i)
            tma_load_2d_pair(dst + i * kBoxBytes, &maps.xp, bar, t.n0 + rank * half + 64 * i, t.prow0 + kb * 64);
    }
}

// This CTA's 128 rows of the row operand of k-block kb (t: this CTA's half of the tile).
template <int KIND>
__device__ __forceinline__ void load_rows_pair(const TcMaps &maps, const Tile &t, int kb, uint32_t dst, uint32_t bar)
{
    if constexpr (KIND == TcUpGate) {
        tma_load_rows_pair(dst, &maps.xp, &maps.xp128, bar, kb * 64, t.prow0 + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDown) {
        tma_load_rows_pair(dst, &maps.hm, &maps.hm128, bar, 0, t.pbase + kb * t.cp + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDownDgrad) {
        tma_load_rows_pair(dst, &maps.dyp, &maps.dyp128, bar, kb * 64, t.prow0 + t.m0, t.a_boxes);
    } else if constexpr (KIND == TcDownWgrad) {
        for (int i = 0; i < t.a_boxes; ++i) tma_load_2d_pair(dst + i * kBoxBytes, &maps.dyp, bar, t.m0 + 64 * i, t.prow0 + kb * 64);
    } else if constexpr (KIND == TcUpGateDgrad) {
        const int hk = t.h / 64;
        const bool second = kb >= hk;
        const int kk = second ? kb - hk : kb;
        tma_load_rows_pair(dst, second ? &maps.db : &maps.da, second ? &maps.db128 : &maps.da128, bar, 0,
                           t.pbase + kk * t.cp + t.m0, t.a_boxes);
    } else {
        const CUtensorMap *am = t.which ? &maps.db : &maps.da;
        for (int i = 0; i < t.a_boxes; ++i)
            tma_load_2d_pair(dst + i * kBoxBytes, am, bar, 0, t.pbase + (t.m0 / 64 + i) * t.cp + kb * 64);
    }
}

// Tile hand-out inside a pair: the leader's tile warp takes tile after tile from the global counter and writes
// each index into the queue slot of both CTAs (its partner's through the cluster's shared address space, the
// arrival that follows releases it at cluster scope); every consuming role of either CTA frees the slot on the
// leader's barrier.  Consumers: the leader's TMA, MMA and epilogue warps, its partner's TMA and epilogue warps.

__device__ __forceinline__ void hand_out_tiles_pair(const TcParams &prm, SmemTail *st, int total, const WaitCtx &w)
{
    for (int it = 0;; ++it) {
        const int slot = it & (kTileQ - 1);
        const uint32_t ph = (uint32_t)(it / kTileQ) & 1u;
        if (it > 0 && !mbar_wait(smem_u32(&st->tq_taken), (uint32_t)(it - 1) & 1u, w)) return;
        if (!mbar_wait_cluster(smem_u32(&st->tq_empty[slot]), ph ^ 1u, w)) return;
        int tile = atomicAdd(prm.tile_counter, 1);
        if (tile >= total) tile = -1;
        st->tile_q[slot] = tile;
        asm volatile("st.shared::cluster.b32 [%0], %1;" ::"r"(map_to_cta(smem_u32(&st->tile_q[slot]), 1)), "r"(tile) : "memory");
        mbar_arrive(smem_u32(&st->tq_full[slot]));
        mbar_arrive_cluster(map_to_cta(smem_u32(&st->tq_full[slot]), 1));
        if (tile < 0) return;
    }
}

// The it-th tile of this cluster (-1: no more), not yet released.
template <int KIND>
__device__ __forceinline__ int peek_tile_pair(const TcParams &prm, SmemTail *st, int it, int total, int cluster_id,
                                              int n_clusters, const WaitCtx &w, bool &ok)
{
    if (!prm.dynamic) {
        const int tile = dealt_tile<KIND>(it, cluster_id, n_clusters);
        return tile >= total ? -1 : tile;
    }
    const int slot = it & (kTileQ - 1);
    const uint32_t ph = (uint32_t)(it / kTileQ) & 1u;
    if (!mbar_wait_cluster(smem_u32(&st->tq_full[slot]), ph, w)) { ok = false; return -1; }
    return *reinterpret_cast<volatile int *>(&st->tile_q[slot]);
}
__device__ __forceinline__ void release_tile_pair(const TcParams &prm, SmemTail *st, int it)
{
    if (prm.dynamic) mbar_arrive_remote(map_to_cta(smem_u32(&st->tq_empty[it & (kTileQ - 1)]), 0));
}

template <int KIND, int VAR, int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(threads_of<EPI>(), 1)
tc_grouped_gemm_pair(const __grid_constant__ TcMaps maps, const __grid_constant__ TcParams prm)
{
    constexpr int NQ = EPI / 4;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t pad = ((raw + 1023u) & ~1023u) - raw;
    unsigned char *smem = smem_raw + pad;
    const uint32_t stage_base = raw + pad;
    unsigned char *epi_bufs = smem + (size_t)kPairStages * kPairStageBytes;
    SmemTail *st = reinterpret_cast<SmemTail *>(epi_bufs + EPI * kEpiBufBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rank = (int)cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    if (tid == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(smem_u32(&st->full[s]), 1);
            mbar_init(smem_u32(&st->empty[s]), 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(smem_u32(&st->tmem_full[a]), 1);
            mbar_init(smem_u32(&st->tmem_empty[a]), 2 * EPI);      // one lane of every epilogue warp of both CTAs
        }
        mbar_init(smem_u32(&st->tq_taken), 1);
        for (int q = 0; q < kTileQ; ++q) {
            mbar_init(smem_u32(&st->tq_full[q]), 1);
            mbar_init(smem_u32(&st->tq_empty[q]), 3 + 2 * EPI);   // used in the leader only
        }
        st->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    build_schedule<KIND, true>(prm, st, reinterpret_cast<int *>(epi_bufs), reinterpret_cast<int *>(epi_bufs) + kMaxExperts, tid);
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32(&st->tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                 // both CTAs' barriers exist before any remote arrival or copy completion
    tc_fence_after();
    const uint32_t tmem_base = st->tmem_base;
    const int total_tiles = st->tstart[prm.meta.N];
    const WaitCtx wc{&st->abort_flag, prm.status, prm.wait_limit_ns};

    if (warp == 0) {
        // ===================== TMA producer (both CTAs) =====================
        if (lane == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int it = 0; ok; ++it) {
                const int tile = peek_tile_pair<KIND>(prm, st, it, total_tiles, cluster_id, n_clusters, wc, ok);
                if (!ok) break;
                release_tile_pair(prm, st, it);
                if (prm.dynamic && rank == 0) mbar_arrive(smem_u32(&st->tq_taken));
                if (tile < 0 || tile == prm.skip_tile) break;
                const Tile t0 = decode_tile<KIND, true>(prm, st, tile, cursor);
                const Tile mine = rank ? second_half(t0) : t0;
                const uint32_t bytes =
                    (uint32_t)(t0.a_boxes + t0.a_boxes_peer + 2 * (pair_n_mma<KIND>(t0) / 128)) * kBoxBytes;
                for (int kb = 0; kb < t0.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->empty[stage]), phase ^ 1u, wc)) { ok = false; break; }
                    const uint32_t leader_bar = map_to_cta(smem_u32(&st->full[stage]), 0);
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&st->full[stage]), bytes);
                    const uint32_t a_dst = stage_base + stage * kPairStageBytes;
                    load_rows_pair<KIND>(maps, mine, kb, a_dst, leader_bar);
                    load_cols_pair<KIND>(maps, t0, rank, kb, a_dst + kARegion, leader_bar);
                    ++issued;
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok && rank == 0) {
                // the copies of both CTAs complete on the leader's barriers: it lets those in flight land
                const int n = issued < kPairStages ? (int)issued : kPairStages;
                for (int i = 1; i <= n; ++i) {
                    int s2 = stage - i;
                    uint32_t ph = phase;
                    if (s2 < 0) { s2 += kPairStages; ph ^= 1u; }
                    const unsigned long long tb = global_ns();
                    while (!mbar_try_wait(smem_u32(&st->full[s2]), ph) && global_ns() - tb < prm.wait_limit_ns) {}
                }
            }
        }
    } else if (warp == 1) {
        // ===================== MMA issuer (leader only) =====================
        if (lane == 0 && rank == 0) {
            int stage = 0, cursor = 0;
            uint32_t phase = 0;
            bool ok = true;
            constexpr bool a_mn = KindTraits<KIND>::a_mn, b_mn = KindTraits<KIND>::b_mn;
            constexpr uint32_t a_step = a_mn ? (2048u >> 4) : (32u >> 4);
            constexpr uint32_t b_step = b_mn ? (2048u >> 4) : (32u >> 4);
            for (int it = 0; ok; ++it) {
                const int tile = peek_tile_pair<KIND>(prm, st, it, total_tiles, cluster_id, n_clusters, wc, ok);
                if (!ok) break;
                release_tile_pair(prm, st, it);
                if (tile < 0) break;
                const Tile t = decode_tile<KIND, true>(prm, st, tile, cursor);
                const int acc = it & 1;
                const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
                if (!mbar_wait(smem_u32(&st->tmem_empty[acc]), acc_phase ^ 1u, wc)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tacc = tmem_base + (uint32_t)(acc * kAccCols);
                const uint32_t idesc = make_idesc(a_mn, b_mn, pair_n_mma<KIND>(t), 256);
                for (int kb = 0; kb < t.nk; ++kb) {
                    if (!mbar_wait(smem_u32(&st->full[stage]), phase, wc)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = stage_base + stage * kPairStageBytes;
                    const uint64_t adesc = make_desc(a_addr, a_mn);
                    const uint64_t bdesc = make_desc(a_addr + kARegion, b_mn);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16_pair(tacc, adesc + (uint64_t)(ks * a_step), bdesc + (uint64_t)(ks * b_step), idesc,
                                       (kb > 0 || ks > 0) ? 1u : 0u);
                    umma_commit_pair(smem_u32(&st->empty[stage]));
                    if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
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
    } else if (warp == 2) {
        // ===================== tile hand-out (leader only) =====================
        if (lane == 0 && rank == 0 && prm.dynamic) hand_out_tiles_pair(prm, st, total_tiles, wc);
    } else if (warp >= kFirstEpiWarp) {
        // ===================== epilogue (both CTAs) =====================
        const int quad = warp & 3;
        const int cq = (warp - kFirstEpiWarp) >> 2;
        const int row = quad * 32 + lane;
        unsigned char *stg = epi_bufs + (warp - kFirstEpiWarp) * kEpiBufBytes;
        const uint32_t leader_empty0 = map_to_cta(smem_u32(&st->tmem_empty[0]), 0);
        const uint32_t leader_empty1 = map_to_cta(smem_u32(&st->tmem_empty[1]), 0);
        int cursor = 0;
        bool ok = true;
        for (int it = 0; ok; ++it) {
            const int tile = peek_tile_pair<KIND>(prm, st, it, total_tiles, cluster_id, n_clusters, wc, ok);
            if (!ok) break;
            __syncwarp();
            if (lane == 0) release_tile_pair(prm, st, it);
            if (tile < 0) break;
            const Tile t0 = decode_tile<KIND, true>(prm, st, tile, cursor);
            const Tile mine = rank ? second_half(t0) : t0;
            const int acc = it & 1;
            const uint32_t acc_phase = (uint32_t)(it >> 1) & 1u;
            if (!mbar_wait(smem_u32(&st->tmem_full[acc]), acc_phase, wc)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kAccCols);
            if (mine.mrows > 0) epilogue_row<KIND, VAR, NQ>(prm, mine, tacc, row, lane, cq, stg);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(acc ? leader_empty1 : leader_empty0);
        }
    }

    // ---- teardown: neither CTA leaves while its partner may still touch its shared or tensor memory ----
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// Sums the partial row dots of the down dgrad in slot order and divides by the gate:
// dg[t, j] = <dY_t W_down, Hm_row> / g = <dY_t, E_(t,j)>.  One thread per assignment.
__global__ void __launch_bounds__(256)
dg_finish_kernel(LayerMeta m, int Ttok, int Pmax, int per_tile, const int *__restrict__ topk_idx,
                 const float *__restrict__ topk_gate, const int *__restrict__ prow_of, const float *__restrict__ dg_part,
                 float *__restrict__ dg, int *status)
{
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= Ttok * m.k) return;
    const int e = topk_idx[i], prow = prow_of[i];
    if (e < 0 || e >= m.N || prow < 0 || prow >= Pmax) { atomicMax(status, kDevBounds); return; }
    const int slots = per_tile * ((m.hoff[e + 1] - m.hoff[e] + 255) / 256);     // one per epilogue warp of a lane quadrant and 256-column tile
    float acc = 0.f;
    for (int sl = 0; sl < slots; ++sl) acc += dg_part[(size_t)sl * Pmax + prow];
    const float g = topk_gate[i];
    dg[i] = (g > 0.f) ? acc / g : 0.f;
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

// bf16 row-major matrix [rows, cols] seen as a 2-D tensor, boxes of box_cols columns x box_rows rows.
// L2 promotion of 128 bytes: measured 1.5-2 % faster per step than 256 bytes or none (two alternating runs each).
bool encode_2d(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows = 64,
               uint32_t box_cols = 64, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B)
{
    EncodeTiledFn fn = get_encode();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool tc_fill_maps(TcMaps &maps, const LayerMeta &m, const WsLayout &L, const WsPtrs &p, const modse_weights_t *w,
                  const void *x, bool backward)
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
    ok = ok && encode_2d(&maps.xg, x, (uint64_t)L.T, m.d, 1);
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

template <int KIND, bool WIDE, int VAR, int EPI>
cudaError_t launch_one(const TcMaps &maps, const TcParams &prm, int grid, cudaStream_t s, int *launches)
{
    auto kern = tc_grouped_gemm<KIND, WIDE, VAR, EPI>;
    constexpr size_t smem = smem_bytes<WIDE, EPI>();
    // the shared-memory attribute of a kernel is set once per process and device
    static unsigned long long attr_done = 0;      // bit per device ordinal (devices beyond 63 set it every time)
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev > 63 || !((attr_done >> dev) & 1ull)) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev <= 63) attr_done |= 1ull << dev;
    }
    kern<<<grid, threads_of<EPI>(), smem, s>>>(maps, prm);
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

template <int KIND, bool WIDE, int VAR>
cudaError_t launch_epi(const TcMaps &maps, const TcParams &prm, int grid, int epi, cudaStream_t s, int *launches)
{
    return epi == 16 ? launch_one<KIND, WIDE, VAR, 16>(maps, prm, grid, s, launches)
                     : launch_one<KIND, WIDE, VAR, 8>(maps, prm, grid, s, launches);
}

template <int KIND, bool HAS_VAR>
cudaError_t launch_kind(const TcMaps &maps, const TcParams &prm, int grid, bool wide, int var, int epi, cudaStream_t s,
                        int *launches)
{
    if constexpr (HAS_VAR) {
        if (var)
            return wide ? launch_epi<KIND, true, 1>(maps, prm, grid, epi, s, launches)
                        : launch_epi<KIND, false, 1>(maps, prm, grid, epi, s, launches);
    }
    return wide ? launch_epi<KIND, true, 0>(maps, prm, grid, epi, s, launches)
                : launch_epi<KIND, false, 0>(maps, prm, grid, epi, s, launches);
}

template <int KIND, int VAR, int EPI>
cudaError_t launch_pair_one(const TcMaps &maps, const TcParams &prm, int grid, cudaStream_t s, int *launches)
{
    auto kern = tc_grouped_gemm_pair<KIND, VAR, EPI>;
    constexpr size_t smem = pair_smem_bytes<EPI>();
    static unsigned long long attr_done = 0;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev > 63 || !((attr_done >> dev) & 1ull)) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev <= 63) attr_done |= 1ull << dev;
    }
    kern<<<grid & ~1, threads_of<EPI>(), smem, s>>>(maps, prm);     // whole clusters of two
    e = cudaGetLastError();
    if (e == cudaSuccess && launches) ++*launches;
    return e;
}

template <int KIND, bool HAS_VAR>
cudaError_t launch_pair(const TcMaps &maps, const TcParams &prm, int grid, int var, int epi, cudaStream_t s, int *launches)
{
    if constexpr (HAS_VAR) {
        if (var)
            return epi == 16 ? launch_pair_one<KIND, 1, 16>(maps, prm, grid, s, launches)
                             : launch_pair_one<KIND, 1, 8>(maps, prm, grid, s, launches);
    }
    return epi == 16 ? launch_pair_one<KIND, 0, 16>(maps, prm, grid, s, launches)
                     : launch_pair_one<KIND, 0, 8>(maps, prm, grid, s, launches);
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

cudaError_t tc_launch(TcPlan &plan, TcKind kind, const TcMaps &maps, const LayerMeta &m, const WsLayout &L,
                      const WsPtrs &p, const modse_wgrads_t *g, bool save, bool out_f32, int fuse, float *scatter_out,
                      cudaStream_t s, int *launches)
{
    TcParams prm{};
    prm.meta = m;
    prm.poffsets = p.poffsets;
    prm.ebase = p.ebase;
    prm.status = p.status;
    prm.tile_counter = p.status + 4 + (int)kind;
    prm.pgate = p.pgate;
    prm.ptoken_of = p.ptoken_of;
    prm.hm = (__nv_bfloat16 *)p.hm;
    prm.sp = (__nv_bfloat16 *)p.a_pre;
    prm.sq = (__nv_bfloat16 *)p.b_pre;
    prm.da = (__nv_bfloat16 *)p.da;
    prm.db = (__nv_bfloat16 *)p.db;
    prm.o = (float *)p.o;
    prm.dxp = (float *)p.dxp;
    prm.dg_part = p.dg_part;
    prm.scatter_out = scatter_out;
    if (g) {
        prm.dw_gate = (__nv_bfloat16 *)g->dw_gate;
        prm.dw_up = (__nv_bfloat16 *)g->dw_up;
        prm.dw_down = (__nv_bfloat16 *)g->dw_down;
    }
    prm.wait_limit_ns = (unsigned long long)g_wait_limit_ms * 1000000ull;
    prm.Pmax = L.Pmax;
    prm.T = L.T;
    prm.save = save ? 1 : 0;
    prm.out_f32 = out_f32 ? 1 : 0;
    prm.dynamic = g_dynamic_tiles;
    prm.skip_tile = (g_skip_kind == (int)kind) ? g_skip_tile : -1;
    const int grid = sm_count(plan);
    const int mask = plan.tile_mask >= 0 ? plan.tile_mask : tc_default_plan();
    const bool wide = ((mask >> (int)kind) & 1) != 0;
    // the two-CTA kernel has no row-gathering loads: the fused up/gate product stays on one CTA
    const bool pair = ((mask >> (kTcPairShift + (int)kind)) & 1) != 0 && grid >= 2 && !(kind == TcUpGate && (fuse & kFuseGather));
    const int epi = (((pair ? g_epi16_pair : wide ? g_epi16_wide : g_epi16_narrow) >> (int)kind) & 1) ? 16 : 8;
    cudaError_t e = cudaErrorInvalidValue;
    if (pair) {
        switch (kind) {
        case TcUpGate: e = launch_pair<TcUpGate, false>(maps, prm, grid, 0, epi, s, launches); break;
        case TcDown: e = launch_pair<TcDown, true>(maps, prm, grid, fuse & kFuseScatter, epi, s, launches); break;
        case TcDownDgrad: e = launch_pair<TcDownDgrad, true>(maps, prm, grid, fuse & kFuseDgRowdot, epi, s, launches); break;
        case TcDownWgrad: e = launch_pair<TcDownWgrad, false>(maps, prm, grid, 0, epi, s, launches); break;
        case TcUpGateDgrad: e = launch_pair<TcUpGateDgrad, true>(maps, prm, grid, fuse & kFuseScatter, epi, s, launches); break;
        case TcUpGateWgrad: e = launch_pair<TcUpGateWgrad, false>(maps, prm, grid, 0, epi, s, launches); break;
        }
    } else
    switch (kind) {
    case TcUpGate: e = launch_kind<TcUpGate, true>(maps, prm, grid, wide, fuse & kFuseGather, epi, s, launches); break;
    case TcDown: e = launch_kind<TcDown, true>(maps, prm, grid, wide, fuse & kFuseScatter, epi, s, launches); break;
    case TcDownDgrad: e = launch_kind<TcDownDgrad, true>(maps, prm, grid, wide, fuse & kFuseDgRowdot, epi, s, launches); break;
    case TcDownWgrad: e = launch_kind<TcDownWgrad, false>(maps, prm, grid, wide, 0, epi, s, launches); break;
    case TcUpGateDgrad: e = launch_kind<TcUpGateDgrad, true>(maps, prm, grid, wide, fuse & kFuseScatter, epi, s, launches); break;
    case TcUpGateWgrad: e = launch_kind<TcUpGateWgrad, false>(maps, prm, grid, wide, 0, epi, s, launches); break;
    }
    if (e != cudaSuccess) return e;
    if (kind == TcDownDgrad && (fuse & kFuseDgRowdot)) {
        const int n = L.T * m.k;
        dg_finish_kernel<<<(n + 255) / 256, 256, 0, s>>>(m, L.T, L.Pmax, epi / 4, p.topk_idx, p.topk_gate, p.prow_of,
                                                         p.dg_part, p.dg, p.status);
        e = cudaGetLastError();
        if (e == cudaSuccess && launches) ++*launches;
    }
    return e;
}

}  // namespace modse
