// bf16 tensor-core (tcgen05 / TMEM) kernel for the two products of the SBP linear backward (Eq. 5).
//
//   dX tiles:  D[m, i] = sum_j dY[keep_rows[m], j] * W[i, j]            (both operands K-major)
//              A = kept rows of dY, gathered straight from the full dY; B = W tile (TMA);
//              the epilogue rounds to bf16 and writes each row to dX[keep_rows[m], :] (whole 128-byte
//              pieces of four rows per store, through a shared-memory transpose).
//   dW tiles:  D[j, i] = sum_m dY[keep_rows[m], j] * X_keep[m, i]       (both operands MN-major)
//              computed transposed so that the gathered operand is again the 128-row side:
//              A = gathered dY rows, B = X_keep tile (TMA); the epilogue stages 16 x 128 pieces of
//              dW[i, j] and sends them out as TMA stores; long reductions can be cut into pieces
//              whose partials a second kernel adds in order.
//
// ONE persistent kernel runs both products: every CTA (one per SM) walks a static, cost-sorted
// list of 128 x BN output tiles of either kind.  The operand ring (64-deep, 128-byte-swizzled
// stages behind full/empty mbarriers) never drains between tiles, and the fp32 accumulator in
// tensor memory is double-buffered, so the epilogue of one tile overlaps the MMAs of the next.
// Warp roles: warps 0-3 epilogue (TMEM lane quadrant = warp id), warp 4 TMA producer of the dense
// operand, warp 5 MMA issuer and TMEM owner, warps 6-9 gather producers, which copy the indexed
// rows of dY with coalesced 16-byte cp.async into the swizzled layout the MMA reads; each thread's
// copies signal the stage's barrier when they land (cp.async.mbarrier.arrive).  TMA tile::gather4
// was measured at ~45 ns of issue time per instruction per SM whatever it fetches - far too slow
// to feed a tile - and is not used.  Every wait is bounded and reports through the status word.
// Four side warps work next to the pipeline: they write the zeros of the dropped rows of dX for the
// block's dX tiles (ahead of the MMAs, so every row of dX is written exactly once and no memset pass
// is needed), then sum the block's share of the kept rows of dY column-wise for the bias gradient
// and leave one partial row per block for a fixed-order reduce.  The row maps are compile-time
// variants: keep_rows on both sides, or identity on either side for gradients kept packed between
// chained layers (Sec. 3.3.1).
#include <map>
#include <mutex>
#include <tuple>

#include "tc_ptx.cuh"

namespace sbp {
namespace {

constexpr int kGatherWarp0 = 6;          // first gather warp
constexpr int kGatherWarps = 4;          // four: the copy instructions of a stage are issue-bound in two warps (dW tiles: 800 of
                                         // the 880 clocks of a k-block), and 448 threads still leave 128 registers each
constexpr int kGatherThreads = 32 * kGatherWarps;
constexpr int kBiasWarp0 = kGatherWarp0 + kGatherWarps;   // four bias warps ride along after the gather warps
constexpr int kBiasThreads = 128;
constexpr int kTcThreads = 32 * kBiasWarp0 + kBiasThreads;
// Which of the eight warps from kGatherWarp0 on gather and which work on the side.  Plain order (gather 6-9, side 10-13)
// for the wide tiles.  For narrow layers the map is interleaved - gather 6, 7, 10, 11, side 8, 9, 12, 13: a warp's
// scheduler is its number modulo 4, so the gather warps, which issue copies all the time, then share schedulers 2 and 3
// with two epilogue warps only, and the TMA and MMA threads (warps 4 and 5) share theirs with side warps that fall idle
// once the zero rows are written.  Measured on the same GPU: ConvNeXt stage-1 pw1 57.9 -> 52.9 us; the wide variants
// gain nothing from it (ViT-B proj and ConvNeXt stage-2 pw1 lose 4-6 %), so they keep the plain order.
static_assert(kGatherWarps == 4 && kBiasThreads == 128, "the warp maps below are written for 4 + 4 warps");
template <bool kInterleaved> __device__ __forceinline__ bool is_gather_warp(int warp) {
    const int w = warp - kGatherWarp0;
    return w >= 0 && (kInterleaved ? (w & 2) == 0 : w < kGatherWarps);
}
template <bool kInterleaved> __device__ __forceinline__ int gather_index(int warp) {
    const int w = warp - kGatherWarp0;
    return kInterleaved ? (w & 1) + (w >> 2) * 2 : w;
}
template <bool kInterleaved> __device__ __forceinline__ int side_index(int warp) {
    const int w = warp - kGatherWarp0;
    return kInterleaved ? ((w - 2) & 1) + ((w - 2) >> 2) * 2 : w - kGatherWarps;
}
constexpr int kBM = 128;                 // accumulator rows per tile (= TMEM lanes)
constexpr int kBK = 64;                  // reduction depth per stage: 64 bf16 = one 128-byte swizzle row
constexpr uint32_t kUmmaK = 16;          // reduction depth of one tcgen05.mma for 16-bit operands
constexpr uint32_t kRowBytes = 128;      // bytes per swizzled smem row
constexpr uint32_t kAtomBytes = 1024;    // 8 rows x 128 B: one swizzle atom
constexpr uint32_t kBlock64Bytes = 64 * kRowBytes;   // a 64-row slab (MN-major operands: one 64-wide block)
constexpr int kStages = 4;               // ring depth with 256-wide tiles (48 KB stages)
constexpr int kStagesNarrow = 6;         // ... when both tile kinds are 128 wide (32 KB stages): same 192 KB, half as many again in flight
constexpr uint32_t kABytes = kBM * kRowBytes;        // 16 KB
constexpr uint32_t kBBytesMax = 256 * kRowBytes;     // 32 KB
constexpr uint32_t kStageBytes = kABytes + kBBytesMax;
constexpr uint32_t kAccCols = 256;       // TMEM columns per accumulator buffer (two buffers = all 512)
constexpr int kBiasChunk = 64;           // kept rows whose ids the bias warps stage at a time
// 16-byte loads each side-warp thread keeps in flight for the bias sums: a template parameter of the kernel,
// 8 or 16.  The deep queue finishes long row lists in time; with short lists it only takes memory
// bandwidth from the operand copies (ViT-B fc1: 5 us per call), so the host picks per shape.
// cross-row-group sums + staged row ids, padded so that the staging buffers after it start on a 1024-byte boundary
// (one of them holds a swizzled tensor-core operand)
constexpr uint32_t kBiasSmemBytes = kBiasThreads * 8 * sizeof(float) + kBiasChunk * sizeof(int) + 512;
constexpr int kEpiChunk = 16;            // accumulator columns (= rows of dW) per TMA store of the dW epilogue
constexpr int kEpiBufs = 3;              // staging buffers the dW epilogue rotates through
constexpr uint32_t kEpiBufBytes = kEpiChunk * kBM * sizeof(float);   // 8 KB: 16 rows of dW x 128 columns
constexpr int kEpiBarrier = 2;           // named barrier of the four epilogue warps
constexpr uint32_t kRingBytes = kStages * kStageBytes;
static_assert(kRingBytes == kStagesNarrow * (kABytes + 128 * kRowBytes), "both ring shapes fill the same memory");
constexpr uint32_t kSmemBytes = kRingBytes + 256 + kBiasSmemBytes + kEpiBufs * kEpiBufBytes + 1024;   // ring + control + bias + staging + slack
static_assert((256 + kBiasSmemBytes) % 1024 == 0, "staging buffers start on a 1024-byte boundary");
static_assert(kSmemBytes <= 227 * 1024, "shared memory per block");

struct TcControl {
    uint64_t full_bar[kStagesNarrow];    // 1 arrival carrying the TMA byte count + one arrival per gather thread
    uint64_t empty_bar[kStagesNarrow];   // 1 arrival: tcgen05.commit of the MMAs that read the stage
    uint64_t gather_bar[kStagesNarrow];  // pairs of blocks, odd block: one arrival per gather thread (forwarded to the even block)
    uint64_t acc_full[2];          // 1 arrival: all MMAs of the tile in this accumulator have finished
    uint64_t acc_empty[2];         // 4 arrivals: each epilogue warp has read the accumulator out
    uint32_t tmem_slot;
    int abort_flag;
};
static_assert(sizeof(TcControl) <= 256, "control block");

struct TcParams {
    const __nv_bfloat16* dY;
    const int32_t* dy_rows;        // row m of the products reads row dy_rows[m] of dY (nullptr: row m)
    const int32_t* dx_rows;        // ... and writes row dx_rows[m] of dX (nullptr: row m); M = rows of dX
    const int32_t* M_keep_dev;
    int64_t M, M_keep_cap;
    int C_in, C_out;
    __nv_bfloat16* dX;             // nullptr: no dX tiles
    float* dW_out;                 // nullptr: no dW tiles; dW itself or the partial buffer
    int64_t dw_split_stride;       // elements between partial buffers
    int dw_splits;
    int dw_accumulate;             // add into dW_out (only with one split)
    int db_from_mma;               // narrow layers: db comes out of the dW tiles (a column of ones appended to X_keep);
                                   // db_partial is then [dw_splits, C_out]
    float* db_partial;             // nullptr: no bias sums; else [gridDim.x, C_out] per-CTA column sums of kept dY rows
    int dw_ctas;                   // 0: every block walks the one cost-sorted list of both tile kinds; > 0: the first
                                   // dw_ctas blocks take the dW pieces, the others the dX tiles, both sweeping the kept
                                   // rows in the same order (memory-bound layers: see next_tile)
    int32_t* status_word;
};

// ---- the static tile list -------------------------------------------------------------------
struct Schedule {
    uint32_t x_tiles, x_ntiles, x_kb;                 // dX: row tiles x column tiles, k-blocks per tile
    uint32_t w_tiles, w_ctiles, w_kb_total, w_kb_per; // dW: (C_out tiles x C_in tiles x splits), k-blocks per piece
    uint32_t splits;
    bool w_first;                                     // the costlier kind is handed out first
    uint32_t total;
    uint32_t dw_ctas;                                 // role split (see next_tile); 0 = one list for all blocks
    uint32_t x_rtiles, slab_len, slab_full;           // dX row tiles; row tiles per slab (the first slab_full slabs have one more)
};
struct Tile {
    bool is_dw;
    uint32_t row_tile, col_tile;      // dX: kept-row tile, C_in tile; dW: C_out tile (128), C_in tile (BNW)
    uint32_t split, kb_begin, num_kb;
};

// kTM: accumulator rows one worker's tile spans - 128 for a block, 256 for a pair of blocks (each block then takes half)
template <int BNX, int BNW, int kTM>
__device__ __forceinline__ Schedule make_schedule(const TcParams& p, int64_t M_keep) {
    Schedule s;
    s.x_ntiles = (uint32_t)((p.C_in + BNX - 1) / BNX);
    s.x_tiles = (p.dX != nullptr) ? (uint32_t)((M_keep + kTM - 1) / kTM) * s.x_ntiles : 0u;
    s.x_kb = (uint32_t)((p.C_out + kBK - 1) / kBK);
    s.splits = (uint32_t)p.dw_splits;
    s.w_ctiles = (uint32_t)((p.C_in + BNW - 1) / BNW);
    s.w_tiles = (p.dW_out != nullptr) ? (uint32_t)((p.C_out + kTM - 1) / kTM) * s.w_ctiles * s.splits : 0u;
    s.w_kb_total = (uint32_t)((M_keep + kBK - 1) / kBK);
    s.w_kb_per = (s.w_kb_total + s.splits - 1) / s.splits;
    s.w_first = s.w_kb_per >= s.x_kb;
    s.total = s.x_tiles + s.w_tiles;
    s.dw_ctas = (p.dw_ctas > 0 && s.x_tiles > 0 && s.w_tiles > 0 && (uint32_t)p.dw_ctas < gridDim.x) ? (uint32_t)p.dw_ctas : 0u;
    s.x_rtiles = s.x_ntiles ? s.x_tiles / s.x_ntiles : 0u;
    s.slab_len = s.x_rtiles / s.splits;               // slab z holds slab_len (+1 for z < slab_full) consecutive row tiles
    s.slab_full = s.x_rtiles % s.splits;
    return s;
}

__device__ __forceinline__ Tile decode_tile(const Schedule& s, uint32_t q) {
    Tile t;
    const uint32_t first = s.w_first ? s.w_tiles : s.x_tiles;
    t.is_dw = (q < first) == s.w_first;
    const uint32_t idx = (q < first) ? q : q - first;
    if (t.is_dw) {
        t.split = idx % s.splits;
        const uint32_t ij = idx / s.splits;
        t.row_tile = ij / s.w_ctiles;
        t.col_tile = ij % s.w_ctiles;
        t.kb_begin = s.w_kb_per * t.split;
        const uint32_t end = (t.kb_begin + s.w_kb_per < s.w_kb_total) ? t.kb_begin + s.w_kb_per : s.w_kb_total;
        t.num_kb = (end > t.kb_begin) ? end - t.kb_begin : 0u;
    } else {
        t.split = 0;
        t.row_tile = idx / s.x_ntiles;
        t.col_tile = idx % s.x_ntiles;
        t.kb_begin = 0;
        t.num_kb = s.x_kb;
    }
    return t;
}

// CTA b takes list positions b, 2G-1-b, 2G+b, 4G-1-b, ...: with the list sorted by cost this
// evens out the load without any run-time counter.
// (G workers, this one is number b: the blocks of the grid, or its pairs of blocks)
__device__ __forceinline__ uint32_t list_position(uint32_t pass, uint32_t G, uint32_t b) {
    return pass * G + ((pass & 1u) ? (G - 1u - b) : b);
}

// The tile a block works on in its pass-th round, false when it has none left.
// One list (dw_ctas == 0): the cost-sorted list of both kinds, dealt out as list_position says.
// Role split (memory-bound layers): blocks [0, dw_ctas) take the dW pieces - piece `split` reduces over the split-th
// slab of kept rows - and the other blocks take the dX tiles in slab-interleaved order (first row tile of every slab,
// then the second of every slab, ...).  Both groups then move through every slab of kept rows from its start to its
// end at the same time, so each kept row of dY comes from DRAM once: whichever product reaches a row second finds
// it in L2 (and, being served from L2, catches up with the other).
__device__ __forceinline__ bool next_tile(const Schedule& s, uint32_t pass, Tile& t, uint32_t G, uint32_t b) {
    if (s.dw_ctas == 0u) {
        const uint32_t q = list_position(pass, G, b);
        if (q >= s.total) return false;
        t = decode_tile(s, q);
        return true;
    }
    if (b < s.dw_ctas) {
        const uint32_t q = b + pass * s.dw_ctas;
        if (q >= s.w_tiles) return false;
        t = decode_tile(s, s.w_first ? q : s.x_tiles + q);
        return true;
    }
    const uint32_t q = (b - s.dw_ctas) + pass * (G - s.dw_ctas);
    if (q >= s.x_tiles) return false;
    const uint32_t tr = q / s.x_ntiles;               // position of the row tile in the interleaved order
    const uint32_t lim = s.slab_len * s.splits;       // positions below this: every slab still has a tile at this depth
    const uint32_t depth = tr < lim ? tr / s.splits : s.slab_len;
    const uint32_t slab = tr < lim ? tr % s.splits : tr - lim;
    t.is_dw = false;
    t.split = 0;
    t.row_tile = slab * s.slab_len + (slab < s.slab_full ? slab : s.slab_full) + depth;
    t.col_tile = q % s.x_ntiles;
    t.kb_begin = 0;
    t.num_kb = s.x_kb;
    return true;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// position of 16-byte chunk `chunk` of row `row` inside a 128-byte-swizzled slab
__device__ __forceinline__ uint32_t swizzled(uint32_t row, uint32_t chunk) {
    return row * kRowBytes + ((chunk ^ (row & 7u)) << 4);
}

// Zero the dropped rows of dX that belong to quarter `wq` (32 kept rows) of a dX tile, in the tile's
// column strip: from just after the kept row preceding the quarter's first one up to its last kept
// row (to the end of dX if it holds the very last kept row).  The rows are walked in windows of 32; a
// warp-wide OR marks the kept rows of a window, the rest get zeros.  One warp, no other data needed:
// the side warps run this for every dX tile of the block while the tensor pipe works.
// Row lookups of the kernel: with kPacked false both row maps are the keep_rows list (the usual, scattered
// form) and the lookup is a plain load; the packed forms for chained layers allow a null map (row m itself).
// Kept apart at compile time (and, in the usual form, read through one pointer): the extra test and the
// second pointer, small as they are, cost the usual form 5 us on ViT-B fc1.
template <bool kPacked>
__device__ __forceinline__ int32_t map_row(const int32_t* rows, int64_t m) {
    if constexpr (kPacked) return mapped_row(rows, m);
    else return __ldg(rows + m);
}

template <int BNX, bool kPacked>
__device__ __forceinline__ void zero_dropped_rows(const TcParams& p, const Tile& t, int64_t M_keep, int wq, int lane) {
    const int C_in = p.C_in;
    const int n0 = (int)(t.col_tile * BNX);
    const int strip_cols = (C_in - n0 < BNX) ? C_in - n0 : BNX;   // multiple of 8
    const int strip_vecs = strip_cols >> 3;
    const int64_t m0 = (int64_t)t.row_tile * kBM;
    const int64_t m = m0 + wq * 32 + lane;
    const bool valid = m < M_keep;
    const int64_t cur = valid ? (int64_t)map_row<kPacked>(kPacked ? p.dx_rows : p.dy_rows, m) : -1;
    const int64_t prev = (valid && m > 0) ? (int64_t)map_row<kPacked>(kPacked ? p.dx_rows : p.dy_rows, m - 1) : -1;
    const int nvalid = __popc(__ballot_sync(0xffffffffu, valid));
    if (nvalid == 0) return;
    const int64_t lo = __shfl_sync(0xffffffffu, prev, 0) + 1;
    const int64_t last_cur = __shfl_sync(0xffffffffu, cur, nvalid - 1);
    const int64_t hi = (m0 + wq * 32 + nvalid == M_keep) ? p.M : last_cur;
    for (int64_t base = lo; base < hi; base += 32) {
        const int64_t d = cur - base;
        uint32_t todo = ~__reduce_or_sync(0xffffffffu, (valid && d >= 0 && d < 32) ? (1u << d) : 0u);
        if (hi - base < 32) todo &= (1u << (hi - base)) - 1u;
        if (strip_vecs <= 16) {                      // narrow strip: two rows per store instruction
            while (todo) {
                const int b0 = __ffs(todo) - 1;
                todo &= todo - 1u;
                const int b1 = todo ? __ffs(todo) - 1 : -1;
                if (todo) todo &= todo - 1u;
                const int b = (lane < 16) ? b0 : b1;
                const int v = lane & 15;
                if (b >= 0 && v < strip_vecs)
                    ptx::st_global_v4(p.dX + (base + b) * C_in + n0 + v * 8, 0u, 0u, 0u, 0u);
            }
        } else {
            while (todo) {
                const int b = __ffs(todo) - 1;
                todo &= todo - 1u;
                if (lane < strip_vecs)
                    ptx::st_global_v4(p.dX + (base + b) * C_in + n0 + lane * 8, 0u, 0u, 0u, 0u);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// kPair (wide tiles only): the grid is made of clusters of two blocks that share every tile through the two-SM tensor-core
// instructions (tcgen05.mma.cta_group::2, issued by the even block).  A tile then spans 256 accumulator rows, 128 in each
// block - each block gathers, reads out and stores its own half exactly as it would a tile of its own - and the 256
// columns of the dense operand are split: each block loads only 128 of them, and the tensor cores exchange the halves.
// Measured on B200 a one-SM instruction of width 256 takes 171 clocks where the two-SM form takes the ideal 128, and a
// block reads a third less shared memory per k-block (64 KB instead of 96 KB written and read), which is what held the
// one-block form back.  What crosses the pair: the odd block's TMA loads credit their bytes to the even block's `full`
// barrier; its gather lands on a local barrier that its (otherwise idle) warp 5 forwards with one remote arrival;
// tcgen05.commit signals `empty` and `accumulator full` in both blocks at once; the odd block's epilogue warps release an
// accumulator with remote arrivals.  Both blocks meet at a cluster barrier before either leaves.
template <int BNX, int BNW, int kBiasDepth, bool kPacked, bool kPair>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_backward_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                   const __grid_constant__ CUtensorMap map_dw, const TcParams p) {
    // narrow layers (both tile kinds 128 wide) and pairs (half of a 256-wide dense tile per block) move 32 KB per stage:
    // six stages then fill the ring
    constexpr bool kNarrow = BNX <= 128 && BNW <= 128;
    static_assert(!kPair || (BNX == 256 && BNW == 256), "pairs of blocks run the wide tiles only");
    constexpr int kS = (kNarrow || kPair) ? kStagesNarrow : kStages;
    constexpr uint32_t kDenseRows = (kNarrow || kPair) ? 128u : 256u;        // rows of the dense operand a block holds per stage
    constexpr uint32_t kSB = kABytes + kDenseRows * kRowBytes;
    const uint32_t rank = kPair ? ptx::cluster_ctarank() : 0u;                // 0: the block that issues the MMAs
    const uint32_t workers = kPair ? gridDim.x >> 1 : gridDim.x, worker = kPair ? blockIdx.x >> 1 : blockIdx.x;
    extern __shared__ uint8_t smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t raw_addr = ptx::smem_addr(smem_raw);
    const uint32_t ring = (raw_addr + 1023u) & ~1023u;              // swizzle atoms need 1024-byte alignment
    TcControl* ctl = reinterpret_cast<TcControl*>(smem_raw + (ring - raw_addr) + kRingBytes);

    // ---- set-up that needs nothing from earlier kernels: overlaps their tail ----
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < kS; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_bar[s]), 1 + kGatherThreads + (kPair ? 1 : 0));
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_bar[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->gather_bar[s]), kGatherThreads);
        }
        for (int a = 0; a < 2; ++a) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[a]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[a]), kPair ? 8 : 4);
        }
        ctl->abort_flag = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tensormap(&map_w);
        ptx::prefetch_tensormap(&map_x);
    }
    // Narrow layers leave half of each accumulator slot unused, which makes room for the bias gradient as one more
    // output column of the dW tiles: db[j] = sum_m dY[m, j] * 1.  The "column of ones" is a constant 64 x 64 operand
    // block (MN-major, only its first column set) kept in the third staging buffer; a second, 16-wide MMA per k-step
    // multiplies it with the same gathered rows of dY.  Wide layers have no spare columns in a slot, but under the role
    // split a dW block runs a single piece and never touches the second slot, so the column goes there.
    const uint32_t dw_bufs = p.db_from_mma ? kEpiBufs - 1 : kEpiBufs;   // staging buffers left to the dW epilogue
    const uint32_t ones_off = (ring - raw_addr) + kRingBytes + 256 + kBiasSmemBytes + (kEpiBufs - 1) * kEpiBufBytes;
    if (p.db_from_mma) {
        for (uint32_t w = threadIdx.x; w < kBlock64Bytes / 4; w += kTcThreads) {
            const uint32_t row = w >> 5, word = w & 31u;            // 128-byte rows of 32 words; column 0 sits in chunk (row & 7)
            reinterpret_cast<uint32_t*>(smem_raw + ones_off)[w] = (word == ((row & 7u) << 2)) ? 0x00003F80u : 0u;
        }
        ptx::fence_async_proxy();                                    // read by the tensor core (async proxy)
    }
    if (warp == 5) {
        if constexpr (kPair) ptx::tmem_alloc_pair(ptx::smem_addr(&ctl->tmem_slot), 2 * kAccCols);
        else ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_slot), 2 * kAccCols);
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if constexpr (kPair) ptx::cluster_sync_all();                    // the peer's barriers exist before anything is sent to them
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = *reinterpret_cast<volatile uint32_t*>(&ctl->tmem_slot);
    volatile int* abort_flag = &ctl->abort_flag;
    int32_t* status_word = p.status_word;

    pdl_wait();                                                      // from here on global memory is read
    const bool skip_all = status_word != nullptr && *reinterpret_cast<volatile int32_t*>(status_word) != 0;
    const int64_t M_keep = load_m_keep(p.M_keep_dev, p.M_keep_cap);
    const Schedule sched = make_schedule<BNX, BNW, kPair ? 2 * kBM : kBM>(p, M_keep);
    const int C_in = p.C_in, C_out = p.C_out;
    // this block's tile of round `pass`: a pair's tile covers two 128-row tiles, one for each of its blocks
    auto fetch_tile = [&](uint32_t pass, Tile& t) {
        if (!next_tile(sched, pass, t, workers, worker)) return false;
        if constexpr (kPair) t.row_tile = t.row_tile * 2u + rank;
        return true;
    };

    if (skip_all) {
        // an earlier check failed: leave every output untouched
    } else if (warp == 4) {
        // ---------------- TMA producer: the dense operand of every stage ----------------
        if (lane == 0) {
            uint32_t it = 0;                                         // stage uses so far, over all tiles
            bool ok = true;
            for (uint32_t pass = 0; ok; ++pass) {
                Tile t;
                if (!fetch_tile(pass, t)) break;
                for (uint32_t k = 0; k < t.num_kb; ++k, ++it) {
                    const int s = it % kS;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / kS) & 1u) ^ 1u, abort_flag, status_word);
                    if (!ok) break;
                    const uint32_t full = ptx::smem_addr(&ctl->full_bar[s]);
                    const uint32_t a_dst = ring + s * kSB;
                    if constexpr (kPair) {
                        // this block's 128 of the tile's 256 dense rows; the bytes of both blocks are credited to the even
                        // block's barrier, which expects them all
                        const uint32_t full0 = ptx::map_to_cta(full, 0);
                        if (rank == 0) ptx::mbar_arrive_expect_tx(full, 256u * kRowBytes);
                        if (t.is_dw) {
                            const int row0 = (int)((t.kb_begin + k) * kBK), i0 = (int)(t.col_tile * BNW) + (int)rank * 128;
#pragma unroll
                            for (int b = 0; b < 2; ++b)
                                ptx::tma_load_2d_pair(a_dst + kABytes + b * kBlock64Bytes, &map_x, i0 + b * 64, row0, full0);
                        } else {
                            ptx::tma_load_2d_pair(a_dst + kABytes, &map_w, (int)(k * kBK), (int)(t.col_tile * BNX) + (int)rank * 128, full0);
                        }
                    } else if (t.is_dw) {                            // X_keep tile: BNW/64 blocks of 64 columns x 64 kept rows
                        const int row0 = (int)((t.kb_begin + k) * kBK), i0 = (int)(t.col_tile * BNW);
                        ptx::mbar_arrive_expect_tx(full, BNW * kRowBytes);
#pragma unroll
                        for (int b = 0; b < BNW / 64; ++b)
                            ptx::tma_load_2d(a_dst + kABytes + b * kBlock64Bytes, &map_x, i0 + b * 64, row0, full);
                    } else {                                         // W tile: BNX rows x 64 columns
                        ptx::mbar_arrive_expect_tx(full, BNX * kRowBytes);
                        ptx::tma_load_2d(a_dst + kABytes, &map_w, (int)(k * kBK), (int)(t.col_tile * BNX), full);
                    }
                }
            }
            if (!ok && kPair) {   // (pairs: the barrier may be the peer's; a fixed pause, far longer than any copy takes)
                for (int i = 0; i < 64; ++i) __nanosleep(1000);
            } else if (!ok) {   // let the copies already issued land before shared memory goes away
                for (uint32_t j = (it > (uint32_t)kS ? it - kS : 0u); j < it; ++j) {
                    const uint32_t bar = ptx::smem_addr(&ctl->full_bar[j % kS]);
                    for (int spin = 0; spin < (1 << 14); ++spin)
                        if (ptx::mbar_try_wait(bar, (j / kS) & 1u)) break;
                }
            }
        }
        __syncwarp();
    } else if (warp == 5) {
        // ---------------- MMA issuer (of the pair: the even block's) ----------------
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, used = 0;                               // stage uses, accumulator uses
            bool ok = true;
            for (uint32_t pass = 0; ok; ++pass) {
                Tile t;
                if (!fetch_tile(pass, t)) break;
                if (t.num_kb == 0) continue;
                const uint32_t acc = used & 1u;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[acc]), ((used >> 1) & 1u) ^ 1u, abort_flag, status_word);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                // where the bias column accumulates: the unused half of a narrow tile's slot; with wide tiles the other
                // slot, which a block that runs a single dW piece (the role split) never uses
                const uint32_t bias_tmem = kNarrow ? d_tmem + 128u : tmem_base + (acc ^ 1u) * kAccCols;
                // K-major (dX): a 16-deep slice is 32 bytes along the swizzled row, 8-row groups 1024 B apart.
                // MN-major (dW): a 16-deep slice is 16 rows (two atoms); 64-wide blocks of the MN extent 8 KB apart.
                constexpr int kMmaM = kPair ? 2 * kBM : kBM;
                const uint32_t idesc = t.is_dw ? ptx::umma_idesc_bf16(kMmaM, BNW, true, true)
                                               : ptx::umma_idesc_bf16(kMmaM, BNX, false, false);
                const uint32_t k_step = t.is_dw ? kUmmaK * kRowBytes : kUmmaK * 2;
                const uint32_t lbo = t.is_dw ? kBlock64Bytes : 16;
                for (uint32_t k = 0; k < t.num_kb; ++k, ++it) {
                    const int s = it % kS;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_bar[s]), (it / kS) & 1u, abort_flag, status_word);
                    if (!ok) break;
                    ptx::tc_fence_after_sync();
                    ptx::fence_async_proxy();        // the gathered operand was written by cp.async (generic proxy)
                    const uint32_t a_addr = ring + s * kSB, b_addr = a_addr + kABytes;
#pragma unroll
                    for (uint32_t u = 0; u < kBK / kUmmaK; ++u) {
                        const uint64_t da = ptx::umma_desc_sw128(a_addr + u * k_step, lbo, kAtomBytes);
                        const uint64_t db = ptx::umma_desc_sw128(b_addr + u * k_step, lbo, kAtomBytes);
                        if constexpr (kPair) ptx::umma_bf16_pair(d_tmem, da, db, idesc, (k | u) != 0u);
                        else ptx::umma_bf16(d_tmem, da, db, idesc, (k | u) != 0u);
                        if (!kPair && t.is_dw && t.col_tile == 0 && p.db_from_mma) {   // the bias column: 16 more accumulator columns, the first is db
                            const uint64_t d1 = ptx::umma_desc_sw128(raw_addr + ones_off + u * k_step, kBlock64Bytes, kAtomBytes);
                            ptx::umma_bf16(bias_tmem, da, d1, ptx::umma_idesc_bf16(kBM, 16, true, true), (k | u) != 0u);
                        }
                    }
                    // stage reusable once these MMAs retire (pairs: in both blocks)
                    if constexpr (kPair) ptx::umma_commit_pair(ptx::smem_addr(&ctl->empty_bar[s]));
                    else ptx::umma_commit(ptx::smem_addr(&ctl->empty_bar[s]));
                }
                if (ok) {
                    if constexpr (kPair) ptx::umma_commit_pair(ptx::smem_addr(&ctl->acc_full[acc]));
                    else ptx::umma_commit(ptx::smem_addr(&ctl->acc_full[acc]));
                }
                ++used;
            }
        } else if (kPair && lane == 0) {
            // ---------------- odd block of a pair: tell the issuer when this block's gathered rows have landed ----------------
            uint32_t it = 0;
            bool ok = true;
            for (uint32_t pass = 0; ok; ++pass) {
                Tile t;
                if (!fetch_tile(pass, t)) break;
                for (uint32_t k = 0; k < t.num_kb; ++k, ++it) {
                    const int s = it % kS;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->gather_bar[s]), (it / kS) & 1u, abort_flag, status_word);
                    if (!ok) break;
                    ptx::fence_async_proxy();                        // this block's tensor core reads what its cp.async wrote
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_addr(&ctl->full_bar[s]), 0));
                }
            }
        }
        __syncwarp();
    } else if (is_gather_warp<kNarrow>(warp)) {
        // ---------------- gather producers ----------------
        const int gw = gather_index<kNarrow>(warp);
        uint32_t it = 0;
        bool ok = true;
        for (uint32_t pass = 0; ok; ++pass) {
            Tile t;
            if (!fetch_tile(pass, t)) break;
            if (!t.is_dw) {
                // dX tile: 128 kept rows x 128 bytes per stage; one warp instruction moves 4 rows x 128 B
                constexpr int kInstr = 32 / kGatherWarps;
                const uint32_t chunk = lane & 7, sub = lane >> 3;
                const int64_t m0 = (int64_t)t.row_tile * kBM;
                const __nv_bfloat16* src[kInstr];
#pragma unroll
                for (int i = 0; i < kInstr; ++i) {
                    int64_t m = m0 + (gw * kInstr + i) * 4 + sub;
                    if (m >= M_keep) m = M_keep - 1;                  // padding rows of the last tile: never stored
                    src[i] = p.dY + (int64_t)map_row<kPacked>(p.dy_rows, m) * C_out + chunk * 8;
                }
                for (uint32_t k = 0; k < t.num_kb; ++k, ++it) {
                    const int s = it % kS;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / kS) & 1u) ^ 1u, abort_flag, status_word);
                    ok = __all_sync(0xffffffffu, ok);                 // the warp leaves the loop together
                    if (!ok) break;
                    const uint32_t a_dst = ring + s * kSB;
                    const int col = (int)(k * kBK + chunk * 8);
                    const uint32_t bytes = (col < C_out) ? 16u : 0u;  // columns past C_out read as zero
                    const int off = (col < C_out) ? (int)(k * kBK) : 0;
#pragma unroll
                    for (int i = 0; i < kInstr; ++i)
                        ptx::cp_async_16(a_dst + swizzled((gw * kInstr + i) * 4 + sub, chunk), src[i] + off, bytes);
                    // the stage's barrier gets this thread's arrival when the copies above have landed
                    ptx::cp_async_arrive_noinc(ptx::smem_addr(rank == 0 ? &ctl->full_bar[s] : &ctl->gather_bar[s]));
                }
            } else {
                // dW tile: 64 kept rows x 128 columns (256 B) of dY per stage; one warp instruction moves 2 rows
                constexpr int kRows = 64 / kGatherWarps;             // rows of a stage this warp copies
                constexpr int kIdxPerLane = (kRows + 31) / 32;       // row ids each lane holds per stage
                constexpr int kInstr = kRows / 2;
                constexpr int kAhead = 8;                            // row ids are fetched this many stages early
                const uint32_t c = lane & 15;                        // 16-byte chunk within the 256-byte row piece
                const uint32_t sub = lane >> 4;                      // which of the two rows of this instruction
                const int col = (int)(t.row_tile * kBM) + (int)c * 8;
                const bool col_ok = col < C_out;                     // columns past C_out read as zero
                const __nv_bfloat16* col_ptr = p.dY + (col_ok ? col : 0);
                int nxt[kAhead][kIdxPerLane];
                auto fetch_ids = [&](uint32_t k_first) {
#pragma unroll
                    for (int u = 0; u < kAhead; ++u)
#pragma unroll
                        for (int h = 0; h < kIdxPerLane; ++h) {
                            const int64_t mrow = (int64_t)(t.kb_begin + k_first + u) * kBK + gw * kRows + h * 32 + (lane % kRows);
                            nxt[u][h] = (k_first + u < t.num_kb && mrow < M_keep) ? map_row<kPacked>(p.dy_rows, mrow) : -1;
                        }
                };
                fetch_ids(0);
                for (uint32_t k0 = 0; k0 < t.num_kb && ok; k0 += kAhead) {
                    int cur[kAhead][kIdxPerLane];
#pragma unroll
                    for (int u = 0; u < kAhead; ++u)
#pragma unroll
                        for (int h = 0; h < kIdxPerLane; ++h) cur[u][h] = nxt[u][h];
                    fetch_ids(k0 + kAhead);
#pragma unroll
                    for (int u = 0; u < kAhead; ++u) {
                        if (k0 + u >= t.num_kb) break;
                        const int s = it % kS;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty_bar[s]), ((it / kS) & 1u) ^ 1u, abort_flag, status_word);
                        ok = __all_sync(0xffffffffu, ok);
                        if (!ok) break;
                        const uint32_t a_dst = ring + s * kSB;
#pragma unroll
                        for (int i = 0; i < kInstr; ++i) {
                            const int rl = i * 2 + (int)sub;                                  // row within this warp's share
                            const int g = __shfl_sync(0xffffffffu, cur[u][rl >> 5], rl & 31);
                            const bool live = g >= 0 && col_ok;                               // rows past M_keep read as zero
                            ptx::cp_async_16(a_dst + (c >> 3) * kBlock64Bytes + swizzled(gw * kRows + rl, c & 7u),
                                             col_ptr + (live ? (int64_t)g * C_out : 0), live ? 16u : 0u);
                        }
                        ptx::cp_async_arrive_noinc(ptx::smem_addr(rank == 0 ? &ctl->full_bar[s] : &ctl->gather_bar[s]));
                        ++it;
                    }
                }
            }
        }
        ptx::cp_async_wait_all();
    } else if (warp >= kGatherWarp0) {
        // ---------------- side warps: zeros for the dropped rows of dX, then the bias sums ----------------
        if (p.dX != nullptr && M_keep > 0) {
            for (uint32_t pass = 0;; ++pass) {
                Tile t;
                if (!fetch_tile(pass, t)) break;
                if (!t.is_dw) zero_dropped_rows<BNX, kPacked>(p, t, M_keep, side_index<kNarrow>(warp), lane);
            }
        }
        // db partial of this CTA's share of the kept rows
        if (p.db_partial != nullptr && !p.db_from_mma) {
            float* red = reinterpret_cast<float*>(smem_raw + (ring - raw_addr) + kRingBytes + 256);
            const int t = side_index<kNarrow>(warp) * 32 + lane;
            const int V = C_out >> 3;                                  // 16-byte column vectors per row
            int VT = 16;                                               // vectors covered per pass (power of two <= 128)
            while (VT < V && VT < kBiasThreads) VT <<= 1;
            const int RG = kBiasThreads / VT;                          // row groups working on the same columns
            const int cvt = t % VT, rg = t / VT;
            const int64_t rows_per = (M_keep + gridDim.x - 1) / gridDim.x;
            const int64_t m_begin = rows_per * blockIdx.x;
            const int64_t m_end = (m_begin + rows_per < M_keep) ? m_begin + rows_per : M_keep;
            const uint4* dY4 = reinterpret_cast<const uint4*>(p.dY);
            float* out = p.db_partial + (int64_t)blockIdx.x * C_out;
            int* ids = reinterpret_cast<int*>(red + kBiasThreads * 8);  // row ids of the current chunk of kept rows
            for (int cv0 = 0; cv0 < V; cv0 += VT) {
                const int cv = cv0 + cvt;
                float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                for (int64_t mc = m_begin; mc < m_end; mc += kBiasChunk) {
                    // stage the chunk's row ids once, so that the dY loads below depend on no other load
                    if (t < kBiasChunk) ids[t] = (mc + t < m_end) ? map_row<kPacked>(p.dy_rows, mc + t) : -1;
                    asm volatile("bar.sync 1, %0;" ::"n"(kBiasThreads) : "memory");
                    if (cv < V) {
                        for (int r0 = rg; r0 < kBiasChunk; r0 += RG * kBiasDepth) {
                            uint4 v[kBiasDepth];
#pragma unroll
                            for (int u = 0; u < kBiasDepth; ++u) {
                                const int r = r0 + u * RG;
                                const int row = (r < kBiasChunk) ? ids[r] : -1;
                                v[u] = (row >= 0) ? __ldg(dY4 + (int64_t)row * V + cv) : make_uint4(0u, 0u, 0u, 0u);
                            }
#pragma unroll
                            for (int u = 0; u < kBiasDepth; ++u) {
                                const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    acc[2 * e] += __uint_as_float(w[e] << 16);
                                    acc[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                                }
                            }
                        }
                    }
                    asm volatile("bar.sync 1, %0;" ::"n"(kBiasThreads) : "memory");
                }
                // add the row groups in a fixed order
#pragma unroll
                for (int e = 0; e < 8; ++e) red[t * 8 + e] = acc[e];
                asm volatile("bar.sync 1, %0;" ::"n"(kBiasThreads) : "memory");
                if (rg == 0 && cv < V) {
                    float sum[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) sum[e] = 0.f;
                    for (int g = 0; g < RG; ++g)
#pragma unroll
                        for (int e = 0; e < 8; ++e) sum[e] += red[(g * VT + cvt) * 8 + e];
                    float4* o = reinterpret_cast<float4*>(out + (int64_t)cv * 8);
                    o[0] = make_float4(sum[0], sum[1], sum[2], sum[3]);
                    o[1] = make_float4(sum[4], sum[5], sum[6], sum[7]);
                }
                asm volatile("bar.sync 1, %0;" ::"n"(kBiasThreads) : "memory");
            }
        }
    } else {
        // ---------------- epilogue warps ----------------
        if (M_keep == 0 && p.dX != nullptr) {                        // nothing kept: dX is all zeros
            const int64_t vecs = p.M * (int64_t)(C_in / 8);
            for (int64_t v = (int64_t)blockIdx.x * 128 + threadIdx.x; v < vecs; v += (int64_t)gridDim.x * 128)
                ptx::st_global_v4(p.dX + v * 8, 0u, 0u, 0u, 0u);
        }
        uint32_t used = 0, staged = 0;                               // accumulator uses, staging-buffer uses
        bool ok = true;
        for (uint32_t pass = 0; ok; ++pass) {
            Tile t;
            if (!fetch_tile(pass, t)) break;
            const uint32_t acc = used & 1u;
            const uint32_t taddr = tmem_base + acc * kAccCols + ((uint32_t)(warp * 32) << 16);
            if (!t.is_dw) {
                // ---- dX tile: scatter the kept rows (the dropped rows are zeroed by the side warps) ----
                const int n0 = (int)(t.col_tile * BNX);
                const int strip_cols = (C_in - n0 < BNX) ? C_in - n0 : BNX;   // multiple of 8
                const int64_t m0 = (int64_t)t.row_tile * kBM;
                const int64_t m = m0 + warp * 32 + lane;
                const bool valid = m < M_keep;
                const int64_t cur = valid ? (int64_t)map_row<kPacked>(kPacked ? p.dx_rows : p.dy_rows, m) : -1;
                if (lane == 0) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[acc]), (used >> 1) & 1u, abort_flag, status_word);
                if (threadIdx.x == 0) ptx::bulk_wait_read<0>();       // the staging memory is no longer read by TMA stores of a dW tile
                ok = !ptx::bar_or<kEpiBarrier, 128>(!ok);            // the four epilogue warps go on, or give up, together
                if (!ok) break;
                ptx::tc_fence_after_sync();
                // Each lane holds one row of the accumulator, but a store instruction that writes 32
                // different rows costs 32 memory transactions.  So the warp transposes 64 columns at a
                // time through its own 4 KB of (swizzled) shared memory and writes four rows x 128
                // contiguous bytes per instruction.
                uint8_t* wbuf = smem_raw + (ring - raw_addr) + kRingBytes + 256 + kBiasSmemBytes + warp * 4096;
                const int cur32 = valid ? (int)cur : -1;
                const int sub = lane >> 3, ch = lane & 7;
                float va[32], vb[32];
                ptx::tmem_ld_32x32(taddr, va);
                ptx::tmem_ld_32x32(taddr + 32u, vb);
#pragma unroll 1
                for (int c0 = 0; c0 < strip_cols; c0 += 64) {
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float* f = (q < 4) ? &va[q * 8] : &vb[(q - 4) * 8];
                        *reinterpret_cast<uint4*>(wbuf + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                            make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                    }
                    __syncwarp();
                    if (c0 + 64 < strip_cols) {                      // the next 64 columns are read while these are stored
                        ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 64), va);
                        ptx::tmem_ld_32x32(taddr + (uint32_t)(c0 + 96), vb);
                    }
                    const bool col_ok = c0 + ch * 8 < strip_cols;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int r = i * 4 + sub;
                        const int g = __shfl_sync(0xffffffffu, cur32, r);
                        const uint4 pk = *reinterpret_cast<const uint4*>(wbuf + r * 128 + ((ch ^ (r & 7)) << 4));
                        if (g >= 0 && col_ok)
                            ptx::st_global_v4(p.dX + (int64_t)g * C_in + n0 + c0 + ch * 8, pk.x, pk.y, pk.z, pk.w);
                    }
                    __syncwarp();
                }
            } else {
                // ---- dW tile: accumulator row = output column j, accumulator column = output row i ----
                const int j = (int)(t.row_tile * kBM) + warp * 32 + lane;
                const int i0 = (int)(t.col_tile * BNW);
                float* out_col = p.dW_out + (int64_t)t.split * p.dw_split_stride + (int64_t)i0 * C_out + j;
                const bool bias_col = p.db_from_mma && t.col_tile == 0;
                if (t.num_kb == 0) {                                 // a piece without kept rows contributes zero
                    if (!p.dw_accumulate && j < C_out)
                        for (int c0 = 0; c0 < BNW && i0 + c0 < C_in; ++c0) out_col[(int64_t)c0 * C_out] = 0.f;
                    if (bias_col && j < C_out) p.db_partial[(int64_t)t.split * C_out + j] = 0.f;
                    continue;
                }
                if (lane == 0) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[acc]), (used >> 1) & 1u, abort_flag, status_word);
                ok = !ptx::bar_or<kEpiBarrier, 128>(!ok);            // the four epilogue warps go on, or give up, together
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const bool add_in = p.dw_accumulate != 0;
                {
                    // 16 rows of dW x 128 columns at a time: registers -> staging buffer -> one TMA store (or
                    // reduce-add), which clips at the edges of dW.  A buffer is rewritten three chunks later;
                    // the issuing thread has by then waited for all but the newest store to have read theirs.
                    const int j0 = (int)(t.row_tile * kBM);
                    const int live = (C_in - i0 < BNW) ? C_in - i0 : BNW;
                    const int chunks = (live + kEpiChunk - 1) / kEpiChunk;
                    const uint32_t stage_off = (ring - raw_addr) + kRingBytes + 256 + kBiasSmemBytes;
#pragma unroll 1
                    for (int c = 0; c < chunks; ++c, ++staged) {
                        float v[kEpiChunk];
                        ptx::tmem_ld_32x16(taddr + (uint32_t)(c * kEpiChunk), v);
                        ptx::tmem_ld_wait();
                        const uint32_t buf_off = stage_off + (staged % dw_bufs) * kEpiBufBytes;
                        float* buf = reinterpret_cast<float*>(smem_raw + buf_off) + warp * 32 + lane;
#pragma unroll
                        for (int r = 0; r < kEpiChunk; ++r) buf[r * kBM] = v[r];
                        ptx::fence_async_proxy();
                        if (threadIdx.x == 0) {                          // the buffer written next must have been read out
                            if (dw_bufs >= 3) ptx::bulk_wait_read<1>();
                            else ptx::bulk_wait_read<0>();
                        }
                        ptx::bar_named<kEpiBarrier, 128>();
                        if (threadIdx.x == 0 && j0 < C_out) {            // (a pair's second block may hold columns past the end of dW)
                            if (add_in) ptx::tma_reduce_add_3d(&map_dw, raw_addr + buf_off, j0, i0 + c * kEpiChunk, (int)t.split);
                            else ptx::tma_store_3d(&map_dw, raw_addr + buf_off, j0, i0 + c * kEpiChunk, (int)t.split);
                            ptx::bulk_commit();
                        }
                    }
                    if (bias_col) {                                  // accumulator column 128: this piece's share of db
                        float v[kEpiChunk];
                        ptx::tmem_ld_32x16(kNarrow ? taddr + 128u : tmem_base + (acc ^ 1u) * kAccCols + ((uint32_t)(warp * 32) << 16), v);
                        ptx::tmem_ld_wait();
                        if (j < C_out) p.db_partial[(int64_t)t.split * C_out + j] = v[0];
                    }
                }
            }
            // this warp is done with the accumulator: hand it back to the MMA issuer
            ptx::tc_fence_before_sync();
            if (lane == 0) {
                if constexpr (kPair) ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_addr(&ctl->acc_empty[acc]), 0));
                else ptx::mbar_arrive(ptx::smem_addr(&ctl->acc_empty[acc]));
            }
            ++used;
        }
    }
    if (threadIdx.x == 0) ptx::bulk_wait_all();                      // the TMA stores of the dW epilogue have landed
    ptx::tc_fence_before_sync();
    __syncthreads();
    if constexpr (kPair) ptx::cluster_sync_all();                    // neither block leaves while the other may still reach into it
    if (warp == 5) {
        ptx::tc_fence_after_sync();
        if constexpr (kPair) ptx::tmem_dealloc_pair(tmem_base, 2 * kAccCols);
        else ptx::tmem_dealloc(tmem_base, 2 * kAccCols);
    }
}

// --------------------------------------------------------------------------------------------
// host side: tensor maps, the split plan and the launch
// --------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 row-major [rows, cols] matrix, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem_strides,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 [splits, C_in, C_out] output of the dW tiles, box = 1 x 16 rows x 128 columns, no swizzle
bool make_map_dw(CUtensorMap* map, const float* base, int64_t splits, int64_t C_in, int64_t C_out) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)C_out, (cuuint64_t)C_in, (cuuint64_t)splits};
    const cuuint64_t strides[2] = {(cuuint64_t)C_out * 4, (cuuint64_t)C_in * (cuuint64_t)C_out * 4};
    const cuuint32_t box[3] = {(cuuint32_t)kBM, (cuuint32_t)kEpiChunk, 1};
    const cuuint32_t elem_strides[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(base), dims, strides, box, elem_strides,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct Plan {
    int bnx, bnw;          // accumulator width of dX / dW tiles
    int splits;            // pieces each dW tile's reduction over kept rows is cut into
    int dw_ctas;           // role split: blocks given to the dW pieces (0 = one list for all blocks)
    bool pair;             // pairs of blocks share 256-row tiles through the two-SM tensor-core instructions
    int64_t tiles;         // upper bound of the tile count (from the capacity); tiles of pairs when pair is set
};

// Estimated run time of the tile list for a given split count, in units of one dX k-block: the
// longest per-block total under the kernel's own static assignment (block b takes list positions
// b, 2G-1-b, 2G+b, ...), the epilogue of that block's last tile, and the reduce launch that
// splitting costs.  The weights are measured ratios on ViT-B shapes; they only rank candidates.
double estimate_cost(int64_t x_tiles, int64_t x_kb, int64_t w_tiles, int64_t w_kb, int64_t splits, int64_t dw_elems, int64_t workers) {
    constexpr double kDwKb = 1.12;        // a dW k-block (two gathered MN-major operands) relative to a dX one
    constexpr double kTileSwitch = 0.5;   // per tile: pipeline hand-over
    constexpr double kTailDx = 9.0, kTailDw = 6.0;   // exposed epilogue of the last tile
    const int64_t kb_per = (w_kb + splits - 1) / splits;
    const int64_t w_pieces = w_tiles * splits;
    const int64_t total = x_tiles + w_pieces;
    if (total == 0) return 0.0;
    const int64_t G = total < workers ? total : workers;
    const bool w_first = kb_per >= x_kb;
    const int64_t first = w_first ? w_pieces : x_tiles;
    double worst = 0.0;
    for (int64_t b = 0; b < G; ++b) {
        double sum = 0.0, tail = 0.0;
        for (int64_t pass = 0;; ++pass) {
            const int64_t q = pass * G + ((pass & 1) ? (G - 1 - b) : b);
            if (q >= total) break;
            const bool is_dw = (q < first) == w_first;
            if (is_dw) {
                const int64_t split = (q < first ? q : q - first) % splits;
                int64_t n = w_kb - kb_per * split;
                if (n > kb_per) n = kb_per;
                if (n < 0) n = 0;
                sum += kDwKb * (double)n + kTileSwitch;
                tail = kTailDw;
            } else {
                sum += (double)x_kb + kTileSwitch;
                tail = kTailDx;
            }
        }
        if (sum + tail > worst) worst = sum + tail;
    }
    if (splits > 1) worst += 7.0 + (double)(splits + 1) * (double)dw_elems * 4.0 / 1.7e6;   // launch + traffic of the reduce
    return worst;
}

struct PlanKey {
    int64_t cap, ci, co;
    bool dx;
    bool dy_packed;
    bool operator<(const PlanKey& o) const { return std::tie(cap, ci, co, dx, dy_packed) < std::tie(o.cap, o.ci, o.co, o.dx, o.dy_packed); }
};
std::mutex g_plan_mutex;
struct PlanChoice { int splits, dw_ctas; };
std::map<PlanKey, PlanChoice> g_plan_memo;
int64_t g_plan_searches = 0;

// dy_packed: dY holds the kept rows packed (chained layers).  The role split is not taken then: its two groups walk
// addresses a fixed large stride apart, which random kept rows scatter over the memory channels but packed rows do not
// (ConvNeXt stage-1 lower layer of a packed block: 71 us with the split, 62 us without).
Plan make_plan(int64_t M_keep_cap, int64_t C_in, int64_t C_out, bool want_dw, bool want_dx, bool dy_packed) {
    Plan pl;
    pl.bnx = (C_in >= 256) ? 256 : 128;
    pl.bnw = (C_in >= 256) ? 256 : 128;
    int64_t x_tiles = want_dx ? ((M_keep_cap + kBM - 1) / kBM) * ((C_in + pl.bnx - 1) / pl.bnx) : 0;
    const int64_t x_kb = (C_out + kBK - 1) / kBK;
    int64_t w_tiles = want_dw ? ((C_out + kBM - 1) / kBM) * ((C_in + pl.bnw - 1) / pl.bnw) : 0;
    const int64_t w_kb = (M_keep_cap + kBK - 1) / kBK;
    pl.splits = 1;
    pl.dw_ctas = 0;
    // Wide layers with enough work for every pair run as pairs of blocks unless the role split below takes them (the
    // memory-bound layers gain nothing from the faster tensor-core form).  From some 4000 kept rows on the pairs win on
    // every wide shape of the paper's models (ViT-B/16 at 6272 kept rows: backward 63 -> 55 us).  A call for dX alone has
    // no dW pieces to even out its tile list, so there the pairs must fill their waves about as well as single blocks
    // would (6272 kept rows x 768 columns: 75 tiles on 74 pairs, 43 us against 30 us).
    const bool memory_bound = 2.0 * (double)M_keep_cap * (double)(2 * C_in + C_out) / 6.5e12 >=
                              0.75 * 4.0 * (double)M_keep_cap * (double)C_in * (double)C_out / 1.4e15;
    pl.pair = pl.bnx == 256 && pl.bnw == 256 && C_out >= 256 && M_keep_cap >= 4096 && !(want_dw && want_dx && !dy_packed && memory_bound);
    if (pl.pair && !want_dw) {
        const int64_t pair_tiles = ((M_keep_cap + 2 * kBM - 1) / (2 * kBM)) * ((C_in + pl.bnx - 1) / pl.bnx);
        const auto fill = [](int64_t tiles, int64_t workers) { return (double)tiles / (double)((tiles + workers - 1) / workers * workers); };
        pl.pair = fill(pair_tiles, kNumSMs / 2) + 0.1 >= fill(x_tiles, kNumSMs);
    }
    if (pl.pair) {
        x_tiles = want_dx ? ((M_keep_cap + 2 * kBM - 1) / (2 * kBM)) * ((C_in + pl.bnx - 1) / pl.bnx) : 0;
        w_tiles = want_dw ? ((C_out + 2 * kBM - 1) / (2 * kBM)) * ((C_in + pl.bnw - 1) / pl.bnw) : 0;
    }
    const int64_t workers = pl.pair ? kNumSMs / 2 : kNumSMs;
    if (want_dw) {
        // The same answer for the same shape: every shape a process has asked about is remembered (a few
        // dozen bytes per layer shape, never evicted), so a model's layers do not push each other out.
        const PlanKey key{M_keep_cap, C_in, C_out, want_dx, dy_packed};
        bool known = false;
        {
            std::lock_guard<std::mutex> lock(g_plan_mutex);
            const auto it = g_plan_memo.find(key);
            if (it != g_plan_memo.end()) {
                pl.splits = it->second.splits;
                pl.dw_ctas = it->second.dw_ctas;
                known = true;
            }
        }
        if (!known) {
            // Memory-bound layers (thin ConvNeXt stages, the detection map) with both products: split the blocks
            // into a dW group and a dX group that sweep the kept rows together (see next_tile), so that DRAM sees
            // each kept row of dY once.  The groups are sized by the bytes each has to pull into its SMs: the
            // gathered rows of dY and the dense operand once per tile, plus the dX rows written (the row count of
            // dX is not known here; twice the kept rows is assumed, the paper's usual keep ratio).
            const double t_flop = 4.0 * (double)M_keep_cap * (double)C_in * (double)C_out / 1.4e15;
            const double t_mem = 2.0 * (double)M_keep_cap * (double)(2 * C_in + C_out) / 6.5e12;
            bool role_split = false;
            if (!pl.pair && want_dx && !dy_packed && t_mem >= 0.75 * t_flop && w_tiles > 0 && w_tiles <= kNumSMs / 4) {
                const double dy = 2.0 * (double)M_keep_cap * (double)C_out, xk = 2.0 * (double)M_keep_cap * (double)C_in;
                const double w_cols = (double)((C_in + pl.bnw - 1) / pl.bnw), w_rows = (double)((C_out + kBM - 1) / kBM);
                const double bytes_w = dy * w_cols + xk * w_rows;
                const double x_cols = (double)((C_in + pl.bnx - 1) / pl.bnx);
                const double bytes_x = dy * x_cols + (double)x_tiles * (double)pl.bnx * (double)C_out * 2.0 + 2.0 * xk;
                const double target = bytes_w / (bytes_w + bytes_x) * (double)kNumSMs;
                int64_t sp = (int64_t)(target / (double)w_tiles + 0.5);
                const int64_t x_rtiles = (M_keep_cap + kBM - 1) / kBM;
                // worth it only with enough dX tiles per dX block to balance (a short list leaves the groups uneven)
                if (sp >= 2 && w_kb / sp >= 8 && x_rtiles >= sp && w_tiles * sp <= kNumSMs - 16 &&
                    x_tiles >= 8 * (kNumSMs - w_tiles * sp)) {
                    pl.splits = (int)sp;
                    pl.dw_ctas = (int)(w_tiles * sp);
                    role_split = true;
                }
            }
            if (!role_split) {
                int64_t max_s = w_kb < 64 ? w_kb : 64;
                if (max_s < 1) max_s = 1;
                // the search walks every tile: with very many tiles any cut balances, so bound the work
                while (max_s > 1 && (x_tiles + w_tiles * max_s) * max_s > (1 << 22)) max_s /= 2;
                double best = 0.0;
                for (int64_t sp = 1; sp <= max_s; ++sp) {
                    const double c = estimate_cost(x_tiles, x_kb, w_tiles, w_kb, sp, C_in * C_out, workers);
                    if (sp == 1 || c < best * 0.995) { best = c; pl.splits = (int)sp; }
                }
            }
            std::lock_guard<std::mutex> lock(g_plan_mutex);
            g_plan_memo[key] = PlanChoice{pl.splits, pl.dw_ctas};
            ++g_plan_searches;
        }
    }
    pl.tiles = x_tiles + w_tiles * pl.splits;
    return pl;
}

template <int BNX, int BNW, int DEPTH, bool PACKED, bool PAIR>
cudaError_t launch_fused_variant(dim3 grid, cudaStream_t stream, const CUtensorMap& map_w, const CUtensorMap& map_x,
                                 const CUtensorMap& map_dw, const TcParams& prm) {
    const cudaError_t opt = opt_in_dynamic_smem<tc_backward_kernel<BNX, BNW, DEPTH, PACKED, PAIR>>((int)kSmemBytes);
    if (opt != cudaSuccess) return opt;
    if constexpr (PAIR)
        return launch_pdl_cluster(tc_backward_kernel<BNX, BNW, DEPTH, PACKED, PAIR>, grid, dim3(kTcThreads), kSmemBytes, 2u, stream, map_w,
                                  map_x, map_dw, prm);
    else
        return launch_pdl(tc_backward_kernel<BNX, BNW, DEPTH, PACKED, PAIR>, grid, dim3(kTcThreads), kSmemBytes, stream, map_w, map_x,
                          map_dw, prm);
}

template <int BNX, int BNW, int DEPTH, bool PAIR>
cudaError_t launch_fused_depth(dim3 grid, cudaStream_t stream, const CUtensorMap& map_w, const CUtensorMap& map_x,
                               const CUtensorMap& map_dw, const TcParams& prm) {
    const bool packed = prm.dy_rows == nullptr || prm.dx_rows == nullptr;
    return packed ? launch_fused_variant<BNX, BNW, DEPTH, true, PAIR>(grid, stream, map_w, map_x, map_dw, prm)
                  : launch_fused_variant<BNX, BNW, DEPTH, false, PAIR>(grid, stream, map_w, map_x, map_dw, prm);
}

template <int BNX, int BNW, bool PAIR = false>
cudaError_t launch_fused(dim3 grid, cudaStream_t stream, const CUtensorMap& map_w, const CUtensorMap& map_x,
                         const CUtensorMap& map_dw, const TcParams& prm, bool deep_side_queue) {
    return deep_side_queue ? launch_fused_depth<BNX, BNW, 16, PAIR>(grid, stream, map_w, map_x, map_dw, prm)
                           : launch_fused_depth<BNX, BNW, 8, PAIR>(grid, stream, map_w, map_x, map_dw, prm);
}

}  // namespace

int64_t tc_plan_searches() {
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    return g_plan_searches;
}

bool tc_shapes_supported(int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    // every TMA box (64 columns x up to 128/256 rows) must fit inside its matrix
    return M_keep_cap >= 64 && M < (1ll << 31) && C_in >= 128 && C_out >= 128 && C_in % 8 == 0 && C_out % 8 == 0;
}

size_t tc_dw_workspace_bytes(int64_t M_keep_cap, int64_t C_in, int64_t C_out) {
    // the split count depends on which products a call asks for; size for the larger of the two cases
    int s = 1;
    for (int v = 0; v < 4; ++v) {
        const int sv = make_plan(M_keep_cap, C_in, C_out, true, (v & 1) != 0, (v & 2) != 0).splits;
        if (sv > s) s = sv;
    }
    return s > 1 ? (size_t)s * (size_t)C_in * (size_t)C_out * sizeof(float) : 0;
}

int tc_backward_kernel_count(int64_t M_keep_cap, int64_t C_in, int64_t C_out, bool want_dw, bool want_dx,
                             bool want_db, bool dy_packed) {
    if (!want_dw && !want_dx) return 0;
    const bool reduce_dw = want_dw && make_plan(M_keep_cap, C_in, C_out, want_dw, want_dx, dy_packed).splits > 1;
    return 1 + ((reduce_dw || want_db) ? 1 : 0);       // the two reductions share one launch
}

sbp_status launch_tc_backward(const void* X_keep, const void* dY, const void* W, const int32_t* dy_rows,
                              const int32_t* dx_rows, const int32_t* M_keep_dev, int64_t M, int64_t M_keep_cap, int64_t C_in, int64_t C_out,
                              float* dW, bool accumulate, void* dX, float* db, float* workspace, float* db_workspace,
                              int32_t* status_word, cudaStream_t stream) {
    const bool want_dw = dW != nullptr, want_dx = dX != nullptr;
    if (!want_dw && !want_dx) return SBP_OK;
    const Plan pl = make_plan(M_keep_cap, C_in, C_out, want_dw, want_dx, dy_rows == nullptr);
    CUtensorMap map_w, map_x, map_dw;
    // a product that is not requested still gets a valid map (of the other matrix): it is never used
    const void* w_base = want_dx ? W : X_keep;
    const void* x_base = want_dw ? X_keep : W;
    const uint32_t w_box = pl.pair ? (uint32_t)pl.bnx / 2u : (uint32_t)pl.bnx;   // a block of a pair loads half of the tile's rows of W
    if (!make_map(&map_w, w_base, want_dx ? C_in : M_keep_cap, want_dx ? C_out : C_in, want_dx ? w_box : 64u) ||
        !make_map(&map_x, x_base, want_dw ? M_keep_cap : C_in, want_dw ? C_in : C_out, want_dw ? 64u : w_box))
        return SBP_ERR_CUDA;
    TcParams prm;
    prm.dY = static_cast<const __nv_bfloat16*>(dY);
    prm.dy_rows = dy_rows;
    prm.dx_rows = dx_rows;
    prm.M_keep_dev = M_keep_dev;
    prm.M = M;
    prm.M_keep_cap = M_keep_cap;
    prm.C_in = (int)C_in;
    prm.C_out = (int)C_out;
    prm.dX = static_cast<__nv_bfloat16*>(dX);
    prm.dW_out = want_dw ? (pl.splits > 1 ? workspace : dW) : nullptr;
    prm.dw_split_stride = C_in * C_out;
    prm.dw_splits = pl.splits;
    prm.dw_accumulate = (pl.splits == 1 && accumulate) ? 1 : 0;
    // the dW tiles leave through TMA stores: dW and the workspace are 16-byte aligned (checked at the entry point)
    if (want_dw) {
        if (!make_map_dw(&map_dw, prm.dW_out, pl.splits, C_in, C_out)) return SBP_ERR_CUDA;
    } else {
        map_dw = map_x;                                              // never used
    }
    prm.db_partial = (db != nullptr) ? db_workspace : nullptr;
    // narrow layers (both tile kinds 128 wide), and wide ones under the role split (one dW piece per block, so the second
    // accumulator slot is free): db is one more output column of the dW tiles, one partial row per split
    const bool db_from_mma = db != nullptr && want_dw && ((pl.bnx <= 128 && pl.bnw <= 128) || pl.dw_ctas > 0);
    prm.db_from_mma = db_from_mma ? 1 : 0;
    const int db_rows = db_from_mma ? pl.splits : 0;                 // 0: one row per block (set below)
    prm.status_word = status_word;
    prm.dw_ctas = pl.dw_ctas;
    int64_t ctas = pl.tiles < kNumSMs ? pl.tiles : kNumSMs;
    if (ctas < 1) ctas = 1;
    if (pl.pair) {                                                   // pl.tiles counts tiles of pairs
        const int64_t pairs = pl.tiles < kNumSMs / 2 ? (pl.tiles < 1 ? 1 : pl.tiles) : kNumSMs / 2;
        ctas = 2 * pairs;
    }
    const dim3 grid((unsigned)ctas);
    // Bias sums on the side: 16-byte loads per side-warp thread against the time the main loop leaves them
    // (about 1.3 us per batch of loads in flight, 0.45 us per k-block).  The shallow queue is enough when it
    // ends well within the main loop.
    bool deep_side = true;
    if (db != nullptr) {
        const int64_t x_tiles = want_dx ? ((M_keep_cap + kBM - 1) / kBM) * ((C_in + pl.bnx - 1) / pl.bnx) : 0;
        const int64_t w_tiles = want_dw ? ((C_out + kBM - 1) / kBM) * ((C_in + pl.bnw - 1) / pl.bnw) : 0;
        const double kb_total = (double)x_tiles * (double)((C_out + kBK - 1) / kBK) +
                                (double)w_tiles * (double)((M_keep_cap + kBK - 1) / kBK);
        const double loop_us = kb_total / (double)ctas * 0.45;
        const double loads = (double)((M_keep_cap + ctas - 1) / ctas) * (double)(C_out / 8) / (double)kBiasThreads;
        deep_side = loads / 8.0 * 1.3 > 0.6 * loop_us;
    }
    cudaError_t e;
    if (pl.pair) e = launch_fused<256, 256, true>(grid, stream, map_w, map_x, map_dw, prm, deep_side);
    else if (pl.bnx == 256 && pl.bnw == 256) e = launch_fused<256, 256>(grid, stream, map_w, map_x, map_dw, prm, deep_side);
    else if (pl.bnx == 128 && pl.bnw == 256) e = launch_fused<128, 256>(grid, stream, map_w, map_x, map_dw, prm, deep_side);
    else if (pl.bnx == 256 && pl.bnw == 128) e = launch_fused<256, 128>(grid, stream, map_w, map_x, map_dw, prm, deep_side);
    else e = launch_fused<128, 128>(grid, stream, map_w, map_x, map_dw, prm, deep_side);
    if (e != cudaSuccess) return SBP_ERR_CUDA;
    const bool reduce_dw = want_dw && pl.splits > 1, reduce_db = db != nullptr;
    cudaError_t r = cudaSuccess;
    if (reduce_dw && reduce_db)
        r = launch_reduce_partials_pair(workspace, pl.splits, C_in * C_out, dW, db_workspace, db_rows ? db_rows : (int)ctas, C_out, db,
                                        accumulate, status_word, stream);
    else if (reduce_dw)
        r = launch_reduce_partials(workspace, pl.splits, C_in * C_out, dW, accumulate, status_word, stream);
    else if (reduce_db)
        r = launch_reduce_partials(db_workspace, db_rows ? db_rows : (int)ctas, C_out, db, accumulate, status_word, stream);
    if (r != cudaSuccess) return SBP_ERR_CUDA;
    return SBP_OK;
}

}  // namespace sbp
