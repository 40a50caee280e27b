// Tensor-core convolution path of libqtz: 1x1 (GEMM) and 3x3 / stride 1 / pad 1 layers as an
// implicit GEMM on the 5th-generation tensor cores.
//
//   raw[p][n] = sum_k x_Q[p][k] * w_Q[n][k]          tcgen05.mma kind::i8, u8 x s8 -> s32 in TMEM
//   acc       = raw - z_x sum(w_Q) - z_w sum(x_Q) + K_valid z_x z_w + bias_q      (Eq. 5-6)
//   y         = clamp(z_y + ((acc m_n + 2^(r_n - 1)) >> r_n))                     fused epilogue
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      TMA producer: NHWC activation boxes (one shifted box per filter tap; out-of-image
//               pixels arrive as zeros) and K-major weight tiles into a ring of swizzled stages
//   warp 1      MMA issuer: one elected lane issues tcgen05.mma; up to eight accumulators (512 TMEM columns / tile
//               width) are used round robin, so the MMAs run several tiles ahead of the epilogue
//   warps 2..17 epilogue: four groups of four warps (tiles up to 128 columns wide) or two groups of eight; the groups
//               take the CTA's tiles in turn: tcgen05.ld, cross terms, requantise, clamp, pack to uint8 into a
//               rotating set of swizzled staging boxes (optionally the residual add against a shortcut tile that the
//               store lane fetched into the box); the warps signal each filled box on an mbarrier and never wait
//               for one another.  For 4-bit layers the same warps first expand the packed weights into shared memory
//   warp 18     one store lane per group: TMA store of every filled box (which also clips ragged tile edges), box
//               handed back once the store has read it
// Image stems (few channels, wide filters) run as "row-window" layers: a frame of the input padded
// with z_x is staged one contiguous run per filter row (copied by the producer warp's lanes), and the MMA
// reads the overlapping windows of 120 neighbouring output columns straight out of those runs (pad_copy_kernel).
// Zero filling stands for padding, so the -z_x sum(w) term must skip the padded taps as well:
// the weight sums are tabulated per border class (which filter rows / columns are cut) and each
// epilogue thread, owning one output pixel, picks its class.
//
// No cluster multicast is used anywhere.  Every device-side wait is bounded: when its cycle
// budget runs out the kernel records (QTZ_ERR_DEVICE_TIMEOUT, site) in the handle's status word
// and all roles drain and return.
#include <algorithm>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "qtz_add_math.cuh"
#include "qtz_device_util.cuh"
#include "qtz_dw_math.cuh"
#include "qtz_plan.cuh"
#include "qtz_ptx.cuh"

using namespace qtz_ptx;

namespace {

constexpr int kTileM = 128;          // rows of one accumulator (TMEM lanes)
constexpr int kMaxAcc = 8;           // accumulators in TMEM: as many as fit in its 512 columns, at most eight
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 16;        // epilogue warps: four groups of four or two groups of eight
constexpr int kEpiGroups = 4;        // most epilogue groups; the groups take tiles in turn, so their drains overlap
constexpr int kStoreWarp = 2 + kEpiWarps;            // its lane g issues the output stores of group g
constexpr int kThreadsTc = 32 * (kStoreWarp + 1);    // producer warp, MMA warp, epilogue warps, store warp
constexpr int kMaxObuf = 4;
constexpr int kMaxStages = 8;
constexpr int kDwWarps = 8;          // fused depthwise -> pointwise: epilogue warps 2..9 compute the depthwise layer instead
constexpr int kDwinStages = 2;       // ... from a ring of this many input tiles
constexpr int kNumBarriers = 2 * kMaxStages + 2 * kMaxAcc + 2 * kEpiGroups * kMaxObuf + 1 + 2 * kDwinStages;
constexpr int kResidentBMax = 80 * 1024;   // weights of a whole layer stay in shared memory up to this size
constexpr int kResidentB4Max = 128 * 1024; // ... and up to this size when they arrive as packed 4-bit codes
constexpr int kMaxCls = 16;
constexpr int kRunBytes = 2048;      // row-window layers: bytes of a frame row one copy brings in (256 elements of 8 bytes)
constexpr int kRunCols = 120;        // ... and the output columns of a tile: 16 * 119 + rb <= 2048 for rb <= 128
constexpr int kSmemBudget = 227 * 1024 - 1024;  // leave room for the 1 KB alignment slack

// Division of a 31-bit unsigned number by a constant known on the host, as one high multiply and one
// shift (round-up reciprocal: q = (n * ceil(2^p / d)) >> p with p = 31 + ceil(log2 d), exact for n < 2^31).
struct FastDiv {
    uint32_t mul, shr, d;
};

__host__ inline FastDiv make_fastdiv(uint32_t d)
{
    FastDiv f{0u, 0u, d};
    if (d > 1) {
        uint32_t lg = 0;
        while ((1ull << lg) < d) ++lg;
        const uint32_t p = 31 + lg;
        f.mul = static_cast<uint32_t>(((1ull << p) + d - 1) / d);
        f.shr = p - 32;
    }
    return f;
}

__device__ __forceinline__ uint32_t fdiv(uint32_t n, const FastDiv& f)
{
    return f.d > 1 ? (__umulhi(n, f.mul) >> f.shr) : n;
}

// A 3x3 depthwise layer computed in front of a pointwise layer inside the same kernel (Section 7 recommends fusing
// operators; the intermediate tensor of a depthwise-separable block then never leaves the SM).  A tile is a box of
// tw x th x tb output pixels; for every K block of the pointwise layer (a chunk of BK depthwise channels) the producer
// brings the box of input pixels with its halo into shared memory, eight warps compute the depthwise outputs of the
// chunk, requantise them to the codes of the intermediate tensor (exactly what the stand-alone depthwise kernel
// stores) and write them as the swizzled activation K block the tensor cores read.
struct DwFront {
    const uint32_t* taps;   // [3][tap_pitch]: per filter row and channel, bytes (k0, k1, k2, 0) as int8
    const int32_t* wsum;
    const int32_t* bias;
    const int32_t* mult;
    const int32_t* rshift;
    int32_t tap_pitch, c, h, w;             // channels and extent of the depthwise input
    int32_t zx, zy, act_min, act_max;       // its zero point; quantizer and clamp of the intermediate tensor
    int32_t twin, thin;                     // input columns / rows of a tile
    uint32_t stage_bytes, stage_stride;     // one input tile in the ring
    int32_t gp, pairs, spi, rps, items;     // thread mapping: channel groups, column pairs, row slots per image, rows per slot
};

struct TcArgs {
    FastDiv dv_per_group, dv_group_m, dv_group_last, dv_tiles_w, dv_tiles_h;
    int32_t is4d;
    int32_t tw, th, tb, rows;               // pixel box of one tile and its row count (<= 128)
    int32_t tiles_w, tiles_h, n_tiles;
    int32_t m_tiles, group_m;               // rasterisation: groups of group_m pixel tiles x all n tiles
    uint32_t num_tiles;
    int32_t W, H, B;                        // output extent (2-D case: W = number of pixels)
    int32_t taps, kw, pad, cstride;          // cstride > 0: row-window layer with that convolution stride (else 0)
    // Thread copies (lsu != 0, row-window layers): the lanes of the producer warp bring the frame runs of a tile in
    // with 16-byte asynchronous copies instead of the copy engine, which is the full stage of these layers.
    // src = the frame; full_count: arrivals a ring stage's "full" barrier expects.
    const uint8_t* src;
    int32_t lsu, full_count;
    int64_t frame_row;                       // row-window layers: row pitch of the padded frame, its rows per image,
    int32_t frame_rows, seg_bytes;           // and the bytes of a frame row one tile takes
    int32_t a_blk;                           // bytes of one activation K block in the ring (0: 128 rows of BK bytes)
    // Row-window layers with few output channels compute rrows consecutive output rows in one tile: the weight matrix
    // holds rrows copies of the layer side by side (bn_row columns each), copy r shifted down by r * cstride frame rows,
    // so that every frame row of the tile is multiplied once against all the output rows it feeds.  Column j of the
    // accumulator is then channel j % bn_row of output row h0 + j / bn_row, and staging box r (bn_row bytes wide) is
    // output row h0 + r.  (rrows = 1: an ordinary tile.)
    int32_t rrows, bn_row;
    int32_t kb_per_tap, c_pad;
    int32_t BK, BN, N, out_box, stages, groups;   // groups: epilogue groups in use (1 or 2)
    int32_t obuf;                           // staging boxes per epilogue group (1..4)
    int32_t bres;                           // weight K blocks kept resident in shared memory (0: weights go through the ring)
    const uint8_t* w4;                      // non-NULL: the resident weights arrive as packed 4-bit codes [n_pad][w4_row] (two per byte
    int32_t w4_row;                         // along K) and the epilogue warps expand them to int8 in shared memory before the first tile
    int32_t spb;                            // K blocks per ring stage (one barrier handshake covers them all)
    int32_t n_acc, acc_stride;              // accumulators in TMEM and the columns between them
    int32_t gwarps;                         // warps per epilogue group: 4 (up to four groups) or 8 (up to two)
    uint32_t idesc;
    const int32_t* bias;
    const int32_t* wsum;                    // [ncls][N]
    const int32_t* mult;
    const int32_t* rshift;
    const int32_t* xsum;                    // per input pixel channel sums (only when zw != 0)
    int32_t ncls;
    int32_t kvalid[kMaxCls];
    int32_t zx, zw, zy, act_min, act_max, raw, fast_requant, fold;
    int32_t* y_raw;
    int32_t* status;
    long long wait_budget;
    // Fused residual add (Section 3.2.1): the convolution's own output code t (quantizer zy / act_min / act_max
    // above) is never stored; the shortcut tile s is brought into the output staging box by the store lane, and
    // the epilogue replaces it in place by clamp(z_y + ((t - z_t) m_t + (s - z_s) m_s + 2^(r-1)) >> r).
    // CTA pairs (pointwise layers with wide tiles and a long reduction): two CTAs of a cluster work on one tile of
    // 256 pixels x BN columns.  Each loads its own 128 pixel rows and its half of the weight tile (both CTAs' copies
    // are counted on the first CTA's "full" barriers); the first CTA issues tcgen05.mma.cta_group::2 over both CTAs'
    // shared memory (every weight K block is fetched from L2 by one of the two only), its commits arrive on both
    // CTAs' barriers, and each CTA drains its own 128 accumulator rows.
    int32_t pair;
    int32_t res;                            // 0: plain convolution
    int32_t res_kind;                       // arithmetic form of the add by its shift (see qtz_add_math.cuh)
    qtz_add::AddRule res_rule;
    qtz_add::AddSplit res_split;
    int64_t res_addend;
    DwFront dw;                             // used by the kernels instantiated with a depthwise front only
};

struct SmemLayout {
    uint32_t a_off, b_off, out_off, tbl_off, tbl_stride, mult_rel, sh_rel, addhi_rel, dwin_off, bar_off, total;
    uint32_t a_stage, b_stage, a_blk, b_blk;
};

// Operand ring (activations, and weights unless all `bres` weight blocks of the layer stay resident),
// output staging boxes and one set of per-channel tables per epilogue group, barriers.
__host__ __device__ inline SmemLayout make_layout(int BK, int BN, int stages, int ncls, int out_box, int groups, int obuf, int bres, int spb,
                                                  int a_blk = 0, int pair = 0, uint32_t dwin_bytes = 0)
{
    SmemLayout L;
    L.a_blk = a_blk > 0 ? a_blk : kTileM * BK;   // one K block of activations (row-window layers: one run of the frame) / of weights
    L.b_blk = (pair ? BN / 2 : BN) * BK;         // (a CTA of a pair holds half of the weight tile's columns)
    L.a_stage = (spb * L.a_blk + 1023u) & ~1023u;   // a ring stage holds spb consecutive K blocks; swizzled tiles behind the ring need 1 KB alignment
    L.b_stage = spb * L.b_blk;
    L.a_off = 0;
    L.b_off = L.a_off + stages * L.a_stage;
    L.out_off = L.b_off + (bres > 0 ? bres * L.b_blk : stages * L.b_stage);
    L.tbl_off = L.out_off + groups * obuf * kTileM * out_box;
    L.mult_rel = ncls > 1 ? ncls * BN * 4 : BN * 8;   // first table: [ncls][BN] int32, or [BN] int64 when folded
    L.sh_rel = L.mult_rel + BN * 4;
    L.addhi_rel = L.sh_rel + BN * 4;
    L.tbl_stride = L.addhi_rel + BN * 4;
    L.dwin_off = (L.tbl_off + groups * L.tbl_stride + 127u) & ~127u;   // ring of depthwise input tiles (fused front only)
    L.bar_off = L.dwin_off + dwin_bytes;
    L.total = L.bar_off + kNumBarriers * 8 + 16;
    return L;
}

// d = (c << 16) | (sat_u8(a) << 8) | sat_u8(b)
__device__ __forceinline__ uint32_t pack_sat_u8(int32_t a, int32_t b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

__device__ __forceinline__ void report_timeout(int32_t* status, int site)
{
    if (atomicCAS(status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) status[1] = site;
}

// Swizzled byte offset of (row, col) inside a staging box whose rows are `box` bytes long
// (32, 64 or 128): the 16-byte chunk index is XORed with the low bits of (offset / 128).
__device__ __forceinline__ uint32_t swz(uint32_t row, uint32_t col, uint32_t box)
{
    const uint32_t off = row * box + col;
    return off ^ (((off >> 7) & ((box >> 4) - 1)) << 4);
}

// Requantises 32 accumulator columns of one row and returns them as 8 packed words.
//   kMode 0 (folded):  y - act_min = hi32(acc m + A) >> (r - 32), A = corr m + 2^(r-1) + (z_y - act_min) 2^r
//   kMode 1 (general): the correction (border class, activation sums) is added to acc first
//   kMode 2 (any shift): 64-bit shift and clamp
//   kMode 3 (folded, any shift r >= 1 whose result is known to fit 32 bits): low word of (acc m + A) >> r
template <int kMode, bool kFullRange>
__device__ __forceinline__ void requant32(const uint32_t (&v)[32], const int32_t* __restrict__ mult_s,
                                          const int32_t* __restrict__ sh_s, const int64_t* __restrict__ add64_s,
                                          const int32_t* __restrict__ corr_row, const int32_t* __restrict__ addhi_s,
                                          int32_t rowterm, int32_t span, int32_t off, uint32_t lo4, uint32_t (&packed)[8])
{
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int4 m4 = *reinterpret_cast<const int4*>(mult_s + 4 * q);
        const int4 s4 = *reinterpret_cast<const int4*>(sh_s + 4 * q);
        const int32_t mm[4] = {m4.x, m4.y, m4.z, m4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
        int32_t y[4];
        if (kMode == 0 || kMode == 3) {
            const longlong2 a01 = *reinterpret_cast<const longlong2*>(add64_s + 4 * q);
            const longlong2 a23 = *reinterpret_cast<const longlong2*>(add64_s + 4 * q + 2);
            const int64_t aa[4] = {a01.x, a01.y, a23.x, a23.y};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int64_t prod = static_cast<int64_t>(static_cast<int32_t>(v[4 * q + e])) * mm[e] + aa[e];
                int32_t t;
                if (kMode == 0) {
                    t = static_cast<int32_t>(prod >> 32) >> ss[e];
                } else {
                    // ss = r; the funnel shift stops at 32, the shift by max(r - 32, 0) does the rest
                    const int4 h4 = *reinterpret_cast<const int4*>(addhi_s + 4 * q);
                    const int32_t s2[4] = {h4.x, h4.y, h4.z, h4.w};
                    t = static_cast<int32_t>(__funnelshift_rc(static_cast<uint32_t>(prod), static_cast<uint32_t>(prod >> 32), ss[e])) >> s2[e];
                }
                y[e] = kFullRange ? t : __vimin_s32_relu(t, span);     // [0,255]: the saturating pack clamps
            }
        } else {
            const int4 c4 = *reinterpret_cast<const int4*>(corr_row + 4 * q);
            const int4 h4 = *reinterpret_cast<const int4*>(addhi_s + 4 * q);
            const int32_t cc[4] = {c4.x, c4.y, c4.z, c4.w}, hh[4] = {h4.x, h4.y, h4.z, h4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int32_t full = static_cast<int32_t>(v[4 * q + e]) + cc[e] + rowterm;
                if (kMode == 1) {
                    const int64_t prod = static_cast<int64_t>(full) * mm[e] + (static_cast<int64_t>(hh[e]) << 32);
                    const int32_t t = static_cast<int32_t>(prod >> 32) >> ss[e];
                    y[e] = kFullRange ? t : __vimin_s32_relu(t, span);
                } else {
                    const int64_t prod = static_cast<int64_t>(full) * mm[e] + (static_cast<int64_t>(1) << (ss[e] - 1));
                    const int64_t sh = (prod >> ss[e]) + off;
                    y[e] = static_cast<int32_t>(min(max(sh, static_cast<int64_t>(0)), static_cast<int64_t>(span)));
                }
            }
        }
        packed[q] = pack_sat_u8(y[1], y[0], pack_sat_u8(y[3], y[2], 0u)) + (kFullRange ? 0u : lo4);
    }
}

// Tile order: pixel tiles are taken in groups of group_m; inside a group the pixel tile varies
// fastest, so the CTAs running at the same time share a band of A panels and a band of B panels
// that together fit in L2.
__device__ __forceinline__ void decode_tile(const TcArgs& a, uint32_t tile, uint32_t& m_tile, int& n_tile, uint32_t prank)
{
    if (a.n_tiles == 1) {                   // the usual case for a convolution layer: one column tile
        m_tile = tile;
        n_tile = 0;
    } else {
        const uint32_t g = fdiv(tile, a.dv_per_group), r = tile - g * a.dv_per_group.d;
        const uint32_t m_first = g * static_cast<uint32_t>(a.group_m);
        const bool last = static_cast<uint32_t>(a.m_tiles) - m_first < static_cast<uint32_t>(a.group_m);   // a shorter final group
        const uint32_t q = last ? fdiv(r, a.dv_group_last) : fdiv(r, a.dv_group_m);
        m_tile = m_first + (r - q * (last ? a.dv_group_last.d : a.dv_group_m.d));
        n_tile = static_cast<int>(q);
    }
    // pair mode: the tile is a pair of pixel tiles, this CTA takes the one of its rank
    if (a.pair) m_tile = 2 * m_tile + prank;
}

// First pixel (w0, h0, b0) of pixel tile m_tile.
__device__ __forceinline__ void tile_origin(const TcArgs& a, uint32_t m_tile, int& w0, int& h0, int& b0)
{
    if (a.is4d) {
        const uint32_t q1 = fdiv(m_tile, a.dv_tiles_w);              // m_tile / tiles_w
        const uint32_t q2 = fdiv(q1, a.dv_tiles_h);                   // ... / tiles_h
        w0 = static_cast<int>(m_tile - q1 * a.dv_tiles_w.d) * a.tw;
        h0 = static_cast<int>(q1 - q2 * a.dv_tiles_h.d) * a.th * a.rrows;
        b0 = static_cast<int>(q2) * a.tb;
    } else {
        w0 = static_cast<int>(m_tile) * kTileM;
        h0 = 0;
        b0 = 0;
    }
}

// kPair: the CTA-pair form (launched as clusters of two; it contains cta_group::2 instructions, which a kernel
// launched without clusters must not)
// kFused: 0, or the stride (1 or 2) of a 3x3 depthwise layer computed in front of this pointwise layer (see DwFront)
template <bool kPair, int kFused>
__global__ void __launch_bounds__(kThreadsTc, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_y, const __grid_constant__ CUtensorMap map_s, const TcArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* const smem = smem_raw + (base - smem_u32(smem_raw));
    const SmemLayout L = make_layout(a.BK, a.BN, a.stages, a.ncls, a.out_box, a.groups, a.obuf, a.bres, a.spb, a.a_blk, kPair,
                                     kFused != 0 ? kDwinStages * a.dw.stage_stride : 0u);

    const uint32_t bar_full = base + L.bar_off;
    const uint32_t bar_empty = bar_full + 8 * kMaxStages;
    const uint32_t bar_tfull = bar_empty + 8 * kMaxStages;
    const uint32_t bar_tempty = bar_tfull + 8 * kMaxAcc;
    const uint32_t bar_ofull = bar_tempty + 8 * kMaxAcc;                               // [group][box]: box written
    const uint32_t bar_oempty = bar_ofull + 8 * kEpiGroups * kMaxObuf;        // [group][box]: box read by its store
    const uint32_t bar_wres = bar_oempty + 8 * kEpiGroups * kMaxObuf;         // resident weights have landed
    const uint32_t bar_dfull = bar_wres + 8;                                  // [input tile stage]: landed
    const uint32_t bar_dempty = bar_dfull + 8 * kDwinStages;                  // ... read by all depthwise warps
    volatile uint32_t* const tmem_slot =
        reinterpret_cast<volatile uint32_t*>(smem + L.bar_off + kNumBarriers * 8);
    // pair mode: this CTA's place in its pair, and the pair's place among the pairs (tiles are dealt to pairs)
    uint32_t prank = 0u;
    if constexpr (kPair) prank = cluster_ctarank();
    const uint32_t tile0 = kPair ? blockIdx.x >> 1 : blockIdx.x;
    const uint32_t tile_step = kPair ? gridDim.x >> 1 : gridDim.x;
    volatile uint32_t* const abort_flag = tmem_slot + 1;

    // the shuffle tells the compiler that the warp index is the same in all lanes
    const int warp = __shfl_sync(0xffffffffu, static_cast<int>(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(bar_full + 8 * s, a.full_count);
            mbar_init(bar_empty + 8 * s, 1);
        }
        for (int i = 0; i < kMaxAcc; ++i) {
            mbar_init(bar_tfull + 8 * i, 1);
            mbar_init(bar_tempty + 8 * i, kPair ? 2 * a.gwarps : a.gwarps);   // (a pair's accumulator is drained by both CTAs)
        }
        for (int i = 0; i < kEpiGroups * kMaxObuf; ++i) {
            mbar_init(bar_ofull + 8 * i, a.gwarps);
            mbar_init(bar_oempty + 8 * i, 1);
        }
        mbar_init(bar_wres, a.w4 ? kEpiWarps : 1);    // one arrival per expanding warp, or the producer's expect_tx
        for (int s = 0; s < kDwinStages; ++s) {
            mbar_init(bar_dfull + 8 * s, 1);
            mbar_init(bar_dempty + 8 * s, kDwWarps);
        }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        prefetch_tensormap(&map_y);
        if (a.res) prefetch_tensormap(&map_s);
        // the next kernel of the stream may be scheduled as this one's CTAs leave (it waits for this grid before it
        // touches activations: grid_dependency_wait below)
        grid_launch_dependents();
    }
    if (warp == 1) {
        if constexpr (kPair) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync();      // both CTAs' barriers exist before anything arrives on them from the other CTA
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_slot, 0);

    const int kblocks = a.taps * a.kb_per_tap;

    if (warp == 0) {
        // ------------------------------ TMA producer ------------------------------
        // The whole warp runs the loop in step, so every address, coordinate and counter is a
        // warp-uniform value; one elected lane issues the copies.  (Letting a single lane run the loop
        // alone makes each issue pay for moving its operands into uniform registers: hundreds of
        // cycles per K block, which starves layers with a short reduction.)
        const uint32_t S = static_cast<uint32_t>(a.stages);
        const bool wres = a.bres > 0;
        const int b_rows = kPair ? a.BN >> 1 : a.BN;      // weight rows (output channels) this CTA fetches per K block
        const uint32_t tx = static_cast<uint32_t>(a.spb) *
                            static_cast<uint32_t>((a.cstride > 0 ? a.seg_bytes : a.rows * a.BK) + (wres ? 0 : b_rows * a.BK));
        const int nst = kblocks / a.spb;         // ring stages per tile
        uint32_t stage = 0, phase = 0;
        bool failed = false;
        if (wres && a.w4 == nullptr && tile0 < a.num_tiles) {
            // the layer's weights are small: fetch all of their K blocks once, they stay for every tile
            if (elect_one()) {
                mbar_arrive_expect_tx(bar_wres, static_cast<uint32_t>(a.bres) * L.b_blk);
                int blk = 0;
                for (int tap = 0; tap < a.taps; ++tap)
                    for (int kc = 0; kc < a.c_pad; kc += a.BK, ++blk)
                        tma_load_2d(base + L.b_off + blk * L.b_blk, &map_b, bar_wres, tap * a.c_pad + kc, 0);
            }
            __syncwarp();
        }
        // This kernel may have started while the kernel before it in the stream was still running (programmatic
        // dependent launch): everything above touched only the layer's own constants; activations wait.
        grid_dependency_wait();
        if constexpr (kFused != 0) {
            // ---- depthwise front: one input tile (with its halo; cells outside the image arrive as zeros) per K block
            uint32_t ds = 0, dphase = 0;
            for (uint32_t tile = tile0; !failed && tile < a.num_tiles; tile += tile_step) {
                int n_tile, w0, h0, b0;
                uint32_t m_tile;
                decode_tile(a, tile, m_tile, n_tile, prank);
                tile_origin(a, m_tile, w0, h0, b0);
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!__all_sync(0xffffffffu, mbar_wait(bar_dempty + 8 * ds, dphase ^ 1, a.wait_budget, 64u)) || *abort_flag != 0) {
                        failed = true;
                        break;
                    }
                    if (elect_one()) {
                        mbar_arrive_expect_tx(bar_dfull + 8 * ds, a.dw.stage_bytes);
                        tma_load_4d(base + L.dwin_off + ds * a.dw.stage_stride, &map_a, bar_dfull + 8 * ds, kb * a.BK, w0 * kFused - 1,
                                    h0 * kFused - 1, b0);
                    }
                    __syncwarp();
                    if (++ds == kDwinStages) {
                        ds = 0;
                        dphase ^= 1;
                    }
                }
            }
            if (failed) {
                if (lane == 0) {
                    report_timeout(a.status, QTZ_SITE_SMEM_EMPTY);
                    *abort_flag = 1;
                }
                const uint32_t last = ds == 0 ? kDwinStages - 1 : ds - 1;       // the most recent copy gets a bounded time to land
                (void)mbar_wait(bar_dfull + 8 * last, ds == 0 ? dphase ^ 1 : dphase, 20000000LL);
                failed = false;
            }
        }
        // ---- thread copies: every lane copies 16-byte pieces of the stage's activations; a stage is signalled
        // `lag` stages late, once this warp's copies for it have landed and been fenced for the tensor cores
        uint32_t issued = 0, signalled = 0, sig_stage = 0;
        // stages a signal trails its copies by (what may be in flight); two stages short of the ring so that the MMA
        // warp always has signalled stages ahead of it while the producer waits for a free one
        const uint32_t lag = max(1u, min(S - 3u, 6u));
        for (uint32_t tile = tile0; kFused == 0 && a.lsu != 0 && !failed && tile < a.num_tiles; tile += tile_step) {
            int n_tile, w0, h0, b0;
            uint32_t m_tile;
            decode_tile(a, tile, m_tile, n_tile, prank);
            tile_origin(a, m_tile, w0, h0, b0);
            const int nrow = n_tile * a.BN;
            for (int st = 0; st < nst; ++st) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1, a.wait_budget, 64u)) ||
                    *abort_flag != 0) {
                    failed = true;
                    break;
                }
                const uint32_t full = bar_full + 8 * stage;
                if (!wres && elect_one()) {              // the weights still come through the copy engine
                    mbar_arrive_expect_tx(full, static_cast<uint32_t>(a.spb * a.BN * a.BK));
                    for (int j = 0; j < a.spb; ++j)
                        tma_load_2d(base + L.b_off + stage * L.b_stage + j * L.b_blk, &map_b, full, (st * a.spb + j) * a.c_pad, nrow);
                }
                const uint32_t dst_a = base + L.a_off + stage * L.a_stage;
                {                                        // spb filter rows: 2 KB of each frame row, as it lies
                    const uint8_t* run = a.src + (static_cast<int64_t>(b0) * a.frame_rows + h0 * a.cstride + st * a.spb) * a.frame_row +
                                         16 * w0 + 16 * lane;
                    for (int j = 0; j < a.spb; ++j, run += a.frame_row)
#pragma unroll
                        for (int i = 0; i < kRunBytes / 512; ++i) cp_async_16(dst_a + j * kRunBytes + 16 * lane + 512 * i, run + 512 * i);
                }
                cp_async_commit();
                if (++issued > lag) {
                    switch (lag) {                       // all but the `lag` most recent stages of this lane have landed
                    case 1: cp_async_wait<1>(); break;
                    case 2: cp_async_wait<2>(); break;
                    case 3: cp_async_wait<3>(); break;
                    case 4: cp_async_wait<4>(); break;
                    case 5: cp_async_wait<5>(); break;
                    default: cp_async_wait<6>(); break;
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (elect_one()) mbar_arrive(bar_full + 8 * sig_stage);
                    ++signalled;
                    if (++sig_stage == S) sig_stage = 0;
                }
                if (++stage == S) {
                    stage = 0;
                    phase ^= 1;
                }
            }
        }
        if (a.lsu != 0) {                                // the last stages, and nothing in flight when the CTA leaves
            cp_async_wait<0>();
            fence_proxy_async_smem();
            __syncwarp();
            for (; signalled < issued; ++signalled) {
                if (elect_one()) mbar_arrive(bar_full + 8 * sig_stage);
                if (++sig_stage == S) sig_stage = 0;
            }
            __syncwarp();
        }
        for (uint32_t tile = tile0; kFused == 0 && a.lsu == 0 && !failed && tile < a.num_tiles; tile += tile_step) {
            int n_tile, w0, h0, b0;
            uint32_t m_tile;
            decode_tile(a, tile, m_tile, n_tile, prank);
            tile_origin(a, m_tile, w0, h0, b0);
            const int nrow = n_tile * a.BN + static_cast<int>(prank) * b_rows;   // (pair mode: this CTA's half of the columns)
            int tap_x = 0, tap_y = 0, kcol = 0, kc = 0;   // filter tap of the next K block, its first weight column, channel offset
            // row-window layers: the tile is a run of output columns of one output row; filter row tap_y
            // reads frame row h0 * cstride + tap_y from the byte where the window of column w0 starts (16 w0)
            const int frame_x = 2 * w0, frame_y = b0 * a.frame_rows + h0 * a.cstride;   // 8-byte element, frame row
            for (int st = 0; st < nst; ++st) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1, a.wait_budget, 64u)) ||
                    *abort_flag != 0) {
                    failed = true;
                    break;
                }
                const bool leader = elect_one();
                uint32_t full = bar_full + 8 * stage;
                if constexpr (kPair) {
                    // both CTAs' copies are counted on the FIRST CTA's barrier, which its MMA warp waits on
                    if (prank == 0) {
                        if (leader) mbar_arrive_expect_tx(full, 2 * tx);
                    } else {
                        full = mapa_shared(full, 0u);
                    }
                    for (int j = 0; j < a.spb; ++j) {
                        if (leader) {
                            tma_load_2d_pair(base + L.a_off + stage * L.a_stage + j * L.a_blk, &map_a, full, kc, w0);
                            tma_load_2d_pair(base + L.b_off + stage * L.b_stage + j * L.b_blk, &map_b, full, kcol + kc, nrow);
                        }
                        kc += a.BK;
                    }
                    __syncwarp();
                    if (++stage == S) {
                        stage = 0;
                        phase ^= 1;
                    }
                    continue;
                }
                if (leader) mbar_arrive_expect_tx(full, tx);
                for (int j = 0; j < a.spb; ++j) {
                    if (leader) {
                        const uint32_t dst_a = base + L.a_off + stage * L.a_stage + j * L.a_blk;
                        if (a.is4d)
                            if (a.cstride > 0)
                            {   // one copy per ring stage: the runs of its spb consecutive filter rows, 2 KB apart
                                if (j == 0) tma_load_2d(dst_a, &map_a, full, frame_x, frame_y + tap_y);
                            }
                            else
                                tma_load_4d(dst_a, &map_a, full, kc, w0 + tap_x - a.pad, h0 + tap_y - a.pad, b0);
                        else
                            tma_load_2d(dst_a, &map_a, full, kc, w0);
                        if (!wres) tma_load_2d(base + L.b_off + stage * L.b_stage + j * L.b_blk, &map_b, full, kcol + kc, nrow);
                    }
                    kc += a.BK;
                    if (kc == a.c_pad) {             // next filter tap
                        kc = 0;
                        kcol += a.c_pad;
                        if (++tap_x == a.kw) {
                            tap_x = 0;
                            ++tap_y;
                        }
                    }
                }
                __syncwarp();
                if (++stage == S) {
                    stage = 0;
                    phase ^= 1;
                }
            }
        }
        if (failed) {
            if (lane == 0) {
                report_timeout(a.status, QTZ_SITE_SMEM_EMPTY);
                *abort_flag = 1;
            }
            // drain: give the most recent copy (the others were issued before it) a bounded time to land
            // before the CTA exits
            const uint32_t last = stage == 0 ? S - 1 : stage - 1;
            (void)mbar_wait(bar_full + 8 * last, stage == 0 ? phase ^ 1 : phase, 20000000LL);
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer --------------------------------
        // Again the whole warp runs the loop and one elected lane issues, so descriptors and TMEM
        // addresses stay warp-uniform.  Only this warp ever issues MMAs.
        const uint64_t desc_a0 = a.cstride > 0 ? make_sliding_desc(base + L.a_off) : make_kmajor_desc(base + L.a_off, a.BK);
        const uint64_t desc_b0 = make_kmajor_desc(base + L.b_off, a.BK);
        const uint32_t a_step = L.a_stage >> 4, b_step = L.b_stage >> 4;   // descriptor address units
        const uint32_t a_blk = L.a_blk >> 4, b_blk = L.b_blk >> 4;
        const int nst = kblocks / a.spb;         // ring stages per tile
        const int mmas = a.BK / 32;          // each MMA consumes 32 bytes of K: advance 2 x 16 B
        const uint32_t S = static_cast<uint32_t>(a.stages);
        uint32_t stage = 0, phase = 0;
        uint32_t acc = 0, acc_phase = 0;     // accumulators are used round robin
        bool ok = true;
        const bool wres = a.bres > 0;
        if (wres && tile0 < a.num_tiles && !__all_sync(0xffffffffu, mbar_wait(bar_wres, 0, a.wait_budget, 64u))) {
            if (lane == 0) {
                report_timeout(a.status, QTZ_SITE_TMA_FULL);
                *abort_flag = 1;
            }
            ok = false;
        }
        // (the second CTA of a pair issues no MMAs: its copies are counted on the first CTA's barriers, its stages are
        //  freed and its accumulators published by the first CTA's commits, which arrive on both CTAs' barriers)
        for (uint32_t tile = tile0; ok && (!kPair || prank == 0) && tile < a.num_tiles; tile += tile_step) {
            if (!__all_sync(0xffffffffu, kPair ? mbar_wait_cluster(bar_tempty + 8 * acc, acc_phase ^ 1, a.wait_budget, 128u)
                                             : mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1, a.wait_budget, 128u))) {
                if (lane == 0) {
                    report_timeout(a.status, QTZ_SITE_TMEM_EMPTY);
                    *abort_flag = 1;
                }
                break;
            }
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + acc * a.acc_stride;
            for (int st = 0; st < nst; ++st) {
                const bool full = __all_sync(0xffffffffu, kPair ? mbar_wait_cluster(bar_full + 8 * stage, phase, a.wait_budget, 64u)
                                                                : mbar_wait(bar_full + 8 * stage, phase, a.wait_budget, 64u));
                if (!full) {
                    if (lane == 0) {
                        report_timeout(a.status, QTZ_SITE_TMA_FULL);
                        *abort_flag = 1;
                    }
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (elect_one()) {
                    uint64_t da = desc_a0 + stage * a_step;
                    uint64_t db = desc_b0 + (wres ? static_cast<uint32_t>(st * a.spb) * b_blk : stage * b_step);
                    uint32_t accumulate = st > 0 ? 1u : 0u;      // the tile's first MMA overwrites the accumulator
                    if constexpr (kPair) {
                        for (int j = 0; j < a.spb; ++j, da += a_blk, db += b_blk) {
                            mma_i8_pair(d_tmem, da, db, a.idesc, accumulate);
                            if (mmas >= 2) mma_i8_pair(d_tmem, da + 2, db + 2, a.idesc, 1u);
                            if (mmas == 4) {
                                mma_i8_pair(d_tmem, da + 4, db + 4, a.idesc, 1u);
                                mma_i8_pair(d_tmem, da + 6, db + 6, a.idesc, 1u);
                            }
                            accumulate = 1u;
                        }
                        mma_commit_pair(bar_empty + 8 * stage);              // frees the stage in both CTAs
                        if (st == nst - 1) mma_commit_pair(bar_tfull + 8 * acc);
                    } else {
                        for (int j = 0; j < a.spb; ++j, da += a_blk, db += b_blk) {
                            mma_i8(d_tmem, da, db, a.idesc, accumulate);
                            if (mmas >= 2) mma_i8(d_tmem, da + 2, db + 2, a.idesc, 1u);
                            if (mmas == 4) {
                                mma_i8(d_tmem, da + 4, db + 4, a.idesc, 1u);
                                mma_i8(d_tmem, da + 6, db + 6, a.idesc, 1u);
                            }
                            accumulate = 1u;
                        }
                        mma_commit(bar_empty + 8 * stage);                     // frees the stage once these MMAs have read it
                        if (st == nst - 1) mma_commit(bar_tfull + 8 * acc);
                    }
                }
                __syncwarp();
                if (++stage == S) {
                    stage = 0;
                    phase ^= 1;
                }
            }
            if (++acc == static_cast<uint32_t>(a.n_acc)) {
                acc = 0;
                acc_phase ^= 1;
            }
        }
    } else if (warp == kStoreWarp) {
        // ------------------------------ output stores ------------------------------
        // One lane per epilogue group turns filled staging boxes into TMA stores and hands each box
        // back once its store has read it, so the warps doing arithmetic never wait on a store.
        const int grp = lane;
        grid_dependency_wait();          // the output may alias a buffer the previous kernel still reads; so may the shortcut
        if (grp < a.groups && !a.raw) {
            const uint32_t box_bytes = kTileM * a.out_box;
            const uint32_t out_addr = base + L.out_off + grp * a.obuf * box_bytes;
            const uint32_t ofull = bar_ofull + 8 * kMaxObuf * grp, oempty = bar_oempty + 8 * kMaxObuf * grp;
            const bool lag = a.obuf >= 3;            // release a box one store late: its read is long over by then
            // the boxes of this group's tiles, in the order the epilogue fills them
            struct BoxIter {
                uint32_t tile;
                int nn, left, w0, h0, b0, bx;     // bx: index of the box in its tile (several output rows per tile: the row)
            };
            auto enter_tile = [&](BoxIter& it) {
                // (a column tile that lies wholly beyond the real channels has no box at all: skip it)
                for (; it.tile < a.num_tiles; it.tile += a.groups * tile_step) {
                    int n_tile;
                    uint32_t m_tile;
                    decode_tile(a, it.tile, m_tile, n_tile, prank);
                    it.nn = n_tile * a.BN;
                    it.left = a.BN;
                    it.bx = 0;
                    if (it.nn >= a.N) continue;
                    tile_origin(a, m_tile, it.w0, it.h0, it.b0);
                    return;
                }
            };
            auto advance = [&](BoxIter& it) {
                it.nn += a.out_box;
                it.left -= a.out_box;
                ++it.bx;
                if (a.rrows > 1 ? it.bx >= a.rrows : !(it.left > 0 && it.nn < a.N)) {
                    it.tile += a.groups * tile_step;
                    enter_tile(it);
                }
            };
            // with a fused residual add a box is handed to the epilogue by the arrival of its shortcut tile: the
            // "empty" barrier of the box carries the bytes of that copy
            auto fetch_shortcut = [&](uint32_t slot_, const BoxIter& it) {
                mbar_arrive_expect_tx(oempty + 8 * slot_, static_cast<uint32_t>(a.rows * a.out_box));   // a box has a.rows rows
                if (a.rrows > 1)
                    tma_load_4d(out_addr + slot_ * box_bytes, &map_s, oempty + 8 * slot_, 0, it.w0, it.h0 + it.bx, it.b0);
                else if (a.is4d)
                    tma_load_4d(out_addr + slot_ * box_bytes, &map_s, oempty + 8 * slot_, it.nn, it.w0, it.h0, it.b0);
                else
                    tma_load_2d(out_addr + slot_ * box_bytes, &map_s, oempty + 8 * slot_, it.nn, it.w0);
            };
            BoxIter cur{tile0 + grp * tile_step, 0, 0, 0, 0, 0, 0};
            enter_tile(cur);
            BoxIter ahead = cur;
            if (a.res)
                for (uint32_t i = 0; i < static_cast<uint32_t>(a.obuf) && ahead.tile < a.num_tiles; ++i) {
                    fetch_shortcut(i, ahead);
                    advance(ahead);
                }
            auto release = [&](uint32_t slot_) {
                if (!a.res) {
                    mbar_arrive(oempty + 8 * slot_);
                } else if (ahead.tile < a.num_tiles) {
                    fetch_shortcut(slot_, ahead);
                    advance(ahead);
                }
            };
            uint32_t slot = 0, phase = 0, prev_slot = 0;
            bool have_prev = false;
            while (cur.tile < a.num_tiles) {
                if (!mbar_wait(ofull + 8 * slot, phase, a.wait_budget, 128u)) {
                    report_timeout(a.status, QTZ_SITE_OUT_FULL);
                    *abort_flag = 1;
                    break;
                }
                if (a.rrows > 1)       // (rows past the image's last are clipped by the store)
                    tma_store_4d(&map_y, out_addr + slot * box_bytes, 0, cur.w0, cur.h0 + cur.bx, cur.b0);
                else if (a.is4d)
                    tma_store_4d(&map_y, out_addr + slot * box_bytes, cur.nn, cur.w0, cur.h0, cur.b0);
                else
                    tma_store_2d(&map_y, out_addr + slot * box_bytes, cur.nn, cur.w0);
                tma_store_commit();
                if (lag) {
                    if (have_prev) {
                        tma_store_wait_read_n<1>();
                        release(prev_slot);
                    }
                    prev_slot = slot;
                    have_prev = true;
                } else {
                    tma_store_wait_read();
                    release(slot);
                }
                if (++slot == static_cast<uint32_t>(a.obuf)) {
                    slot = 0;
                    phase ^= 1;
                }
                advance(cur);
            }
            tma_store_wait_all();
        }
    } else if (kFused != 0 && warp >= 2 && warp < 2 + kDwWarps) {
        // ------------------------------ depthwise front ----------------------------
        // Eight warps turn every input tile of the ring into one activation K block.  A piece of work is 4 channels x
        // 2 adjacent output columns x rps output rows (as in the stand-alone depthwise kernel: three byte-transposed
        // input rows rotate through registers, a filter row is one dp4a); the lanes of a warp take neighbouring channel
        // groups, so the reads of the tile and the writes of the K block run along shared-memory rows.
        if constexpr (kFused != 0) {
            using namespace qtz_dw;
            const DwFront& f = a.dw;
            const int wt = threadIdx.x - 64;                 // 0 .. 255
            const int cb = a.BK;
            const uint32_t row_bytes = static_cast<uint32_t>(f.twin * cb);
            WinOffsets wo;
            wo.o1 = cb; wo.o2 = 2 * cb; wo.o3 = 3 * cb; wo.o4 = 4 * cb;
            ChanConst<kModeFast> k;
            k.off = f.zy - f.act_min;
            k.span = f.act_max - f.act_min;
            k.lo4 = 0x01010101u * static_cast<uint32_t>(f.act_min);
            k.zw = 0;
            const uint32_t fill = 0x01010101u * static_cast<uint32_t>(f.zx);
            const uint32_t S = static_cast<uint32_t>(a.stages);
            uint32_t stage = 0, phase = 0, ds = 0, dphase = 0;
            int loaded_c0 = -1;
            bool ok = true;
            for (uint32_t tile = tile0; ok && tile < a.num_tiles; tile += tile_step) {
                int n_tile, w0, h0, b0;
                uint32_t m_tile;
                decode_tile(a, tile, m_tile, n_tile, prank);
                tile_origin(a, m_tile, w0, h0, b0);
                const int ih0 = h0 * kFused - 1, iw0 = w0 * kFused - 1;
                const bool border = f.zx != 0 && (ih0 < 0 || iw0 < 0 || ih0 + f.thin > f.h || iw0 + f.twin > f.w);
                for (int kb = 0; kb < kblocks; ++kb) {
                    // the input tile has landed and the K block's place in the ring is free
                    bool got = __all_sync(0xffffffffu, mbar_wait(bar_dfull + 8 * ds, dphase, a.wait_budget, 64u)) &&
                               __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * stage, phase ^ 1, a.wait_budget, 64u));
                    // (a tile that needs its padding refilled has a barrier among these warps below: they decide
                    //  together, so that no warp is left alone at it when another one's wait ran out)
                    if (border) got = named_barrier_and(9, 32 * kDwWarps, got);
                    if (!got) {
                        if (lane == 0) {
                            report_timeout(a.status, QTZ_SITE_TMA_FULL);
                            *abort_flag = 1;
                        }
                        ok = false;
                        break;
                    }
                    uint8_t* const tile_s = smem + L.dwin_off + ds * f.stage_stride;
                    if (border) {
                        // padding is real zero = the code z_x: overwrite the cells that lie outside the image
                        const int rows_in = min(f.thin, f.h - ih0), first_row = ih0 < 0 ? 1 : 0;
                        const int cols_in = min(f.twin, f.w - iw0), first_col = iw0 < 0 ? 1 : 0;
                        const int lane8 = 8 * lane, warp_id = wt >> 5;
                        for (int img = 0; img < a.tb; ++img) {
                            uint8_t* const img_s = tile_s + img * f.thin * row_bytes;
                            if (first_row)
                                for (uint32_t i = 8 * wt; i < row_bytes; i += 8 * 32 * kDwWarps) *reinterpret_cast<uint2*>(img_s + i) = make_uint2(fill, fill);
                            for (int ri = rows_in; ri < f.thin; ++ri)
                                for (uint32_t i = 8 * wt; i < row_bytes; i += 8 * 32 * kDwWarps)
                                    *reinterpret_cast<uint2*>(img_s + ri * row_bytes + i) = make_uint2(fill, fill);
                            if (first_col + f.twin - cols_in > 0) {
                                for (int ri = first_row + warp_id; ri < rows_in; ri += kDwWarps) {
                                    uint8_t* const row = img_s + ri * row_bytes;
                                    if (first_col)
                                        for (int i = lane8; i < cb; i += 256) *reinterpret_cast<uint2*>(row + i) = make_uint2(fill, fill);
                                    for (int i = lane8; i < (f.twin - cols_in) * cb; i += 256)
                                        *reinterpret_cast<uint2*>(row + cols_in * cb + i) = make_uint2(fill, fill);
                                }
                            }
                        }
                        named_barrier(8, 32 * kDwWarps);
                    }
                    uint8_t* const a_stage = smem + L.a_off + stage * L.a_stage;
                    const uint32_t tile_addr = base + L.dwin_off + ds * f.stage_stride;
                    for (int item = wt; item < f.items; item += 32 * kDwWarps) {
                        const int g = item % f.gp, rest = item / f.gp;
                        const int pr = rest % f.pairs, slot = rest / f.pairs;
                        const int img = slot / f.spi, part = slot - img * f.spi;
                        const int c0 = kb * cb + 4 * g;
                        const int ow0 = 2 * pr;
                        const bool second = ow0 + 1 < a.tw;
                        const int r_begin = part * f.rps;
                        int n = min(a.th, r_begin + f.rps) - r_begin;            // output rows of this piece
                        if (n <= 0) continue;
                        uint32_t arow = static_cast<uint32_t>((img * a.th + r_begin) * a.tw + ow0);   // row of the K block: the tile's pixel
                        if (c0 >= f.c) {                                           // channels beyond the layer's: zero codes
                            for (; n > 0; --n, arow += a.tw) {
                                *reinterpret_cast<uint32_t*>(a_stage + swz(arow, 4 * g, cb)) = 0u;
                                if (second) *reinterpret_cast<uint32_t*>(a_stage + swz(arow + 1, 4 * g, cb)) = 0u;
                            }
                            continue;
                        }
                        // per-channel constants of the piece's four channels (kept while the thread stays on them)
                        if (c0 != loaded_c0) {
                        loaded_c0 = c0;
#pragma unroll
                        for (int i = 0; i < 3; ++i) {
                            const uint4 w = __ldg(reinterpret_cast<const uint4*>(f.taps + static_cast<int64_t>(i) * f.tap_pitch + c0));
                            k.wa[i][0] = w.x; k.wa[i][1] = w.y; k.wa[i][2] = w.z; k.wa[i][3] = w.w;
#pragma unroll
                            for (int ch = 0; ch < 4; ++ch) k.wb[i][ch] = k.wa[i][ch] << 8;
                        }
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            const int32_t r = __ldg(f.rshift + c0 + ch);
                            const int32_t bse = __ldg(f.bias + c0 + ch) - f.zx * __ldg(f.wsum + c0 + ch);
                            k.m[ch] = __ldg(f.mult + c0 + ch);
                            k.sh[ch] = r - 32;
                            k.add[ch] = (static_cast<int64_t>(2 * k.off + 1) << (r - 1)) + static_cast<int64_t>(bse) * k.m[ch];
                        }
                        }
                        auto emit = [&](const RowState<kFused>& r0, const RowState<kFused>& r1, const RowState<kFused>& r2) {
                            int32_t acc[2][4];
                            mac3<kFused, false, kModeFast>(r0, r1, r2, k, acc);
                            const uint32_t y0 = requant_pixel<kModeFast, true>(acc[0], k);
                            const uint32_t y1 = requant_pixel<kModeFast, true>(acc[1], k);
                            *reinterpret_cast<uint32_t*>(a_stage + swz(arow, 4 * g, cb)) = y0;
                            if (second) *reinterpret_cast<uint32_t*>(a_stage + swz(arow + 1, 4 * g, cb)) = y1;
                            arow += a.tw;
                        };
                        uint32_t cell = tile_addr + ((img * f.thin + r_begin * kFused) * f.twin + ow0 * kFused) * cb + 4 * g;
                        if constexpr (kFused == 1) {
                            RowState<1> r0, r1, r2;
                            load_row<1>(cell, wo, r0); cell += row_bytes;
                            load_row<1>(cell, wo, r1); cell += row_bytes;
                            for (; n >= 3; n -= 3) {
                                load_row<1>(cell, wo, r2); cell += row_bytes;
                                emit(r0, r1, r2);
                                load_row<1>(cell, wo, r0); cell += row_bytes;
                                emit(r1, r2, r0);
                                load_row<1>(cell, wo, r1); cell += row_bytes;
                                emit(r2, r0, r1);
                            }
                            if (n >= 1) {
                                load_row<1>(cell, wo, r2); cell += row_bytes;
                                emit(r0, r1, r2);
                                if (n == 2) {
                                    load_row<1>(cell, wo, r0);
                                    emit(r1, r2, r0);
                                }
                            }
                        } else {
                            RowState<2> top, mid, bot;
                            load_row<2>(cell, wo, top); cell += row_bytes;
                            for (; n >= 2; n -= 2) {
                                load_row<2>(cell, wo, mid); cell += row_bytes;
                                load_row<2>(cell, wo, bot); cell += row_bytes;
                                emit(top, mid, bot);
                                load_row<2>(cell, wo, mid); cell += row_bytes;
                                load_row<2>(cell, wo, top); cell += row_bytes;
                                emit(bot, mid, top);
                            }
                            if (n == 1) {
                                load_row<2>(cell, wo, mid); cell += row_bytes;
                                load_row<2>(cell, wo, bot);
                                emit(top, mid, bot);
                            }
                        }
                    }
                    // the K block is written (generic proxy) for the tensor cores (async proxy); the input tile is free
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(bar_full + 8 * stage);
                        mbar_arrive(bar_dempty + 8 * ds);
                    }
                    if (++stage == S) {
                        stage = 0;
                        phase ^= 1;
                    }
                    if (++ds == kDwinStages) {
                        ds = 0;
                        dphase ^= 1;
                    }
                }
            }
        }
    } else {
        // ------------------------------ epilogue ----------------------------------
        // Sixteen warps as four groups of four (narrow tiles: more work per warp and tile, so the per-tile
        // bookkeeping weighs less) or two groups of eight.  The groups take this CTA's tiles in turn, so
        // the waits of one overlap with the arithmetic of the others.  Inside a group a thread owns one
        // accumulator row (one output pixel); with eight warps the two warps of a TMEM lane quarter split
        // the columns of every staging box in halves.  The warps of a group run free of one another: a
        // warp waits for a staging box to be empty, fills its part and signals the box's barrier; the
        // group's store lane issues the store once all warps of the group have signalled.
        const int et = threadIdx.x - 64 - (kFused != 0 ? 32 * kDwWarps : 0);   // 0..511 (0..255 behind a depthwise front)
        const int gthreads = 32 * a.gwarps;          // 128 or 256 threads per group
        const int grp = et / gthreads;
        const int gt = et - grp * gthreads;          // thread within the group
        const int quarter = warp & 3;                // TMEM lane quarter this warp may read
        const int halves = a.gwarps >> 2;            // warps sharing a quarter split every box's columns between them
        const int half = (gt >> 7) & (halves - 1);
        const int row = quarter * 32 + lane;         // accumulator row owned by this thread
        uint8_t* const tbl = smem + L.tbl_off + grp * L.tbl_stride;
        int32_t* const corr_s = reinterpret_cast<int32_t*>(tbl);                     // [ncls][BN] (general form)
        int64_t* const add64_s = reinterpret_cast<int64_t*>(tbl);                    // [BN]       (folded form)
        int32_t* const mult_s = reinterpret_cast<int32_t*>(tbl + L.mult_rel);
        int32_t* const sh_s = reinterpret_cast<int32_t*>(tbl + L.sh_rel);
        int32_t* const addhi_s = reinterpret_cast<int32_t*>(tbl + L.addhi_rel);
        const uint32_t box_bytes = kTileM * a.out_box;
        uint8_t* const out_s = smem + L.out_off + grp * a.obuf * box_bytes;          // this group's staging boxes
        const uint32_t ofull = bar_ofull + 8 * kMaxObuf * grp, oempty = bar_oempty + 8 * kMaxObuf * grp;
        uint32_t slot = 0, slot_phase = 0;                                           // box written next
        const int boxes = (a.BN + a.out_box - 1) / a.out_box;
        const int half_cols = max(32, a.out_box / halves);   // 32, 64 or 128 columns per thread and box (a 32-byte box: one of the two warps)
        const int32_t span = a.act_max - a.act_min, off = a.zy - a.act_min;
        const uint32_t lo4 = 0x01010101u * static_cast<uint32_t>(a.act_min);
        const bool fold = a.fold != 0;
        const int mode = a.fold == 1 ? 0 : (a.fold == 2 ? 3 : (a.fast_requant ? 1 : 2));
        const bool full_range = a.act_min == 0 && a.act_max == 255;   // then saturation to a byte is the whole clamp
        const uint32_t bar_tbl = 1 + grp;
        // this thread's pixel inside a tile never changes
        const int dr_w = a.is4d ? row % a.tw : row;
        const int dr_h = a.is4d ? (row / a.tw) % a.th : 0;
        const int dr_b = a.is4d ? row / (a.tw * a.th) : 0;
        int staged_n_tile = -1;
        // the activation sums come from the kernel launched just before this one, which may still be running; raw
        // accumulators are stored by these warps themselves
        if (a.zw != 0 || a.raw) grid_dependency_wait();
        if (a.w4 != nullptr && a.bres > 0 && tile0 < a.num_tiles) {
            // 4-bit weights: the layer's codes stay packed in global memory (two per byte along K); all sixteen
            // epilogue warps expand this CTA's column tile to int8 once, straight into the swizzled K blocks the
            // tensor cores read.  A thread takes 16 packed bytes = 32 codes = two 16-byte chunks of one row.
            int n_tile0;
            uint32_t m_tile0;
            decode_tile(a, tile0, m_tile0, n_tile0, prank);       // (a CTA with several tiles has a single column tile)
            const int parts = a.BK >> 5;                        // 32-code pieces per row of a K block
            const int per_blk = a.BN * parts;
            const uint8_t* const src = a.w4 + static_cast<int64_t>(n_tile0) * a.BN * a.w4_row;
            for (int q = et; q < a.bres * per_blk; q += 32 * kEpiWarps) {
                const int blk = q / per_blk, rem = q - blk * per_blk;
                const int wrow = rem / parts, part = rem - wrow * parts;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + static_cast<int64_t>(wrow) * a.w4_row + blk * (a.BK >> 1) + 16 * part));
                const uint32_t in[4] = {v.x, v.y, v.z, v.w};
                uint32_t o[8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // byte j of a word holds code 2j (low nibble) and code 2j+1 (high nibble), two's complement
                    uint32_t even = in[i] & 0x0f0f0f0fu, odd = (in[i] >> 4) & 0x0f0f0f0fu;
                    even |= (even & 0x08080808u) * 0x1eu;       // sign bit of a nibble -> bits 4..7 of its byte
                    odd |= (odd & 0x08080808u) * 0x1eu;
                    o[2 * i] = __byte_perm(even, odd, 0x5140);
                    o[2 * i + 1] = __byte_perm(even, odd, 0x7362);
                }
                uint8_t* const dstb = smem + L.b_off + blk * L.b_blk;
                *reinterpret_cast<uint4*>(dstb + swz(wrow, 32 * part, a.BK)) = make_uint4(o[0], o[1], o[2], o[3]);
                *reinterpret_cast<uint4*>(dstb + swz(wrow, 32 * part + 16, a.BK)) = make_uint4(o[4], o[5], o[6], o[7]);
            }
            fence_proxy_async_smem();                           // generic-proxy writes, read next by the tensor cores
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_wres);
        }
        // A warp whose wait ran out stops working but keeps meeting the group at the table barriers,
        // so that nobody is left alone at one; everything else it would have signalled times out too.
        bool dead = false;
        // with two groups in use, group g takes every other tile (accumulator g); with one, group 0 takes all
        // the CTA's i-th tile lives in accumulator i mod n_acc
        uint32_t next_acc = grp % a.n_acc, next_acc_phase = (grp / a.n_acc) & 1;
        uint32_t tile = grp < a.groups ? tile0 + grp * tile_step : a.num_tiles;
        for (; tile < a.num_tiles; tile += a.groups * tile_step) {
            const uint32_t acc = next_acc, acc_phase = next_acc_phase;
            next_acc += a.groups;
            while (next_acc >= static_cast<uint32_t>(a.n_acc)) {
                next_acc -= a.n_acc;
                next_acc_phase ^= 1;
            }
            int n_tile;
            uint32_t m_tile;
            decode_tile(a, tile, m_tile, n_tile, prank);
            const int n0 = n_tile * a.BN;

            if (n_tile != staged_n_tile) {
                // per-channel constants of this column tile: cross-term correction (Eq. 5-6), multiplier,
                // shift, and the rounding constant with the output offset folded in
                named_barrier(bar_tbl, gthreads);            // everyone is done with the old tables
                for (int j = gt; j < a.BN; j += gthreads) {
                    const int n = a.rrows > 1 ? j % a.bn_row : n0 + j;      // (several output rows per tile: the layer's channels repeat)
                    const bool live = n < a.N;
                    const int32_t bias = live ? __ldg(a.bias + n) : 0;
                    const int32_t m = (live && !a.raw) ? __ldg(a.mult + n) : 0;
                    const int32_t r = (live && !a.raw) ? __ldg(a.rshift + n) : 40;
                    const int32_t addhi = a.fast_requant ? (2 * off + 1) * (1 << (r - 33)) : 0;
                    mult_s[j] = m;
                    sh_s[j] = (a.fold == 1 || a.fast_requant) ? r - 32 : r;
                    if (fold) {
                        // rounding constant 2^(r-1) and the output offset (z_y - act_min) 2^r in one 64-bit addend
                        const int32_t ws = live ? __ldg(a.wsum + n) : 0;
                        const int32_t corr = bias - a.zx * ws;
                        add64_s[j] = static_cast<int64_t>(corr) * m + (static_cast<int64_t>(2 * off + 1) << (r - 1));
                        addhi_s[j] = r > 32 ? r - 32 : 0;
                    } else {
                        addhi_s[j] = addhi;
                        for (int c = 0; c < a.ncls; ++c) {
                            const int32_t ws = live ? __ldg(a.wsum + static_cast<int64_t>(c) * a.N + n) : 0;
                            corr_s[c * a.BN + j] = bias - a.zx * ws + a.kvalid[c] * a.zx * a.zw;
                        }
                    }
                }
                staged_n_tile = n_tile;
                named_barrier(bar_tbl, gthreads);            // tables visible to the whole group
            }
            if (dead) continue;

            // which pixel this row is, its border class and its activation-sum term
            int w0, h0, b0;
            tile_origin(a, m_tile, w0, h0, b0);
            const int pw = w0 + dr_w, ph = h0 + dr_h, pb = b0 + dr_b;
            const bool row_live = row < a.rows && pw < a.W && ph < a.H && pb < a.B;
            int cls = 0;
            if (a.ncls > 1) cls = ((ph == 0) | ((ph == a.H - 1) << 1)) * 4 + ((pw == 0) | ((pw == a.W - 1) << 1));
            int32_t rowterm = 0;
            if (a.zw != 0 && row_live) {
                int32_t xs = 0;
                if (a.taps == 1) {
                    xs = __ldg(a.xsum + (static_cast<int64_t>(pb) * a.H + ph) * a.W + pw);
                } else {
                    for (int dy = -1; dy <= 1; ++dy)
                        for (int dx = -1; dx <= 1; ++dx) {
                            const int hh = ph + dy, ww = pw + dx;
                            if (hh >= 0 && hh < a.H && ww >= 0 && ww < a.W)
                                xs += __ldg(a.xsum + (static_cast<int64_t>(pb) * a.H + hh) * a.W + ww);
                        }
                }
                rowterm = -a.zw * xs;
            }
            const int32_t* const corr_row = corr_s + cls * a.BN;

            // every lane polls the accumulator's barrier; the vote keeps the warp's decision uniform
            if (!__all_sync(0xffffffffu, mbar_wait(bar_tfull + 8 * acc, acc_phase, a.wait_budget, 128u))) {
                if (lane == 0) {
                    report_timeout(a.status, QTZ_SITE_TMEM_FULL);
                    *abort_flag = 1;
                }
                dead = true;
                continue;
            }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * a.acc_stride;

            if (a.raw) {
                // int32 accumulators with the cross terms applied; the two warps of a quarter alternate 32-column chunks
                for (int j0 = 32 * half; j0 < a.BN && n0 + j0 < a.N; j0 += 32 * halves) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + j0, v);
                    tmem_ld_wait();
                    if (row_live) {
                        const int64_t pix = a.is4d ? (static_cast<int64_t>(pb) * a.H + ph) * a.W + pw : pw;
                        int32_t* out = a.y_raw + pix * a.N + n0 + j0;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (n0 + j0 + j < a.N) out[j] = static_cast<int32_t>(v[j]) + corr_row[j0 + j] + rowterm;
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (kPair && prank != 0) { if constexpr (kPair) mbar_arrive_remote(bar_tempty + 8 * acc, 0u); }
                    else mbar_arrive(bar_tempty + 8 * acc);
                }
                continue;
            }

            // uint8 output: one staging box (128 rows x out_box bytes) at a time
            for (int bx = 0; bx < boxes; ++bx) {
                // (several output rows per tile: box bx holds all channels of output row h0 + bx)
                const int nn = a.rrows > 1 ? 0 : n0 + bx * a.out_box;
                if (nn >= a.N) break;                // boxes entirely beyond the real channels
                uint8_t* const dst = out_s + slot * box_bytes;
                // the store that last used this box has read it
                // (with a fused residual add this is also the arrival of the shortcut tile in the box: phase k of the
                //  barrier ends when the k-th copy into the box has landed, so the parity to wait for is one earlier)
                if (!__all_sync(0xffffffffu, mbar_wait(oempty + 8 * slot, a.res ? slot_phase : slot_phase ^ 1, a.wait_budget, 64u))) {
                    if (lane == 0) {
                        report_timeout(a.status, QTZ_SITE_OUT_EMPTY);
                        *abort_flag = 1;
                    }
                    dead = true;
                    break;
                }
                for (int col = half * half_cols; col < min((half + 1) * half_cols, a.out_box) && nn + col < a.N; col += 32) {
                    const int j0 = bx * a.out_box + col;
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + j0, v);
                    tmem_ld_wait();
                    uint32_t packed[8];
                    if (mode == 0 && full_range)
                        requant32<0, true>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else if (mode == 0)
                        requant32<0, false>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else if (mode == 3 && full_range)
                        requant32<3, true>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else if (mode == 3)
                        requant32<3, false>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else if (mode == 1 && full_range)
                        requant32<1, true>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else if (mode == 1)
                        requant32<1, false>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    else
                        requant32<2, false>(v, mult_s + j0, sh_s + j0, add64_s + j0, corr_row + j0, addhi_s + j0, rowterm, span, off, lo4, packed);
                    uint4* const p0 = reinterpret_cast<uint4*>(dst + swz(row, col, a.out_box));
                    uint4* const p1 = reinterpret_cast<uint4*>(dst + swz(row, col + 16, a.out_box));
                    if (a.res) {
                        // packed[] holds the convolution's own codes t; the box holds the shortcut s at the same places
                        const uint4 s0 = *p0, s1 = *p1;
                        const uint32_t sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
                        const uint32_t lo4r = 0x01010101u * static_cast<uint32_t>(a.res_rule.act_min);
                        const int32_t spanr = a.res_rule.act_max - a.res_rule.act_min;
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            if (a.res_kind == 3) packed[q] = qtz_add::add_split4(packed[q], sv[q], a.res_split, lo4r);
                            else if (a.res_kind == 0) packed[q] = qtz_add::add4<0>(packed[q], sv[q], a.res_rule, a.res_addend, spanr, lo4r);
                            else if (a.res_kind == 1) packed[q] = qtz_add::add4<1>(packed[q], sv[q], a.res_rule, a.res_addend, spanr, lo4r);
                            else packed[q] = qtz_add::add4<2>(packed[q], sv[q], a.res_rule, a.res_addend, spanr, lo4r);
                        }
                    }
                    *p0 = make_uint4(packed[0], packed[1], packed[2], packed[3]);
                    *p1 = make_uint4(packed[4], packed[5], packed[6], packed[7]);
                }
                const bool drained = bx == boxes - 1 || (a.rrows == 1 && nn + a.out_box >= a.N);
                if (drained) tc_fence_before();
                fence_proxy_async_smem();            // this thread's box writes, for the TMA store
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(ofull + 8 * slot);
                    if (drained) {                                    // accumulator back to the MMA warp (of the pair's first CTA)
                        if (kPair && prank != 0) { if constexpr (kPair) mbar_arrive_remote(bar_tempty + 8 * acc, 0u); }
                        else mbar_arrive(bar_tempty + 8 * acc);
                    }
                }
                if (++slot == static_cast<uint32_t>(a.obuf)) {
                    slot = 0;
                    slot_phase ^= 1;
                }
            }
        }
    }

    if (threadIdx.x == 0) grid_dependency_wait();   // even a CTA without tiles leaves only after the previous grid
    tc_fence_before();
    __syncthreads();
    if constexpr (kPair) cluster_sync();      // the other CTA's MMAs and arrivals no longer touch this CTA's shared memory
    if (warp == 1) {
        tc_fence_after();
        if constexpr (kPair) tmem_dealloc_pair(tmem_base, kTmemCols);
        else tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------
// Preparation kernels (run once per layer) and small pre-passes
// ------------------------------------------------------------------------------------------
constexpr int kPrepThreads = 256;

// OHWI codes -> int8 [n_pad][taps][c_pad], zero padded (K-major rows for the B operand).  The c
// positions of a tap are c / cs runs of cs bytes, of which the first c_src come from the source
// tensor (layers run over an im2col matrix pad every source tap from c_src to cs bytes; otherwise
// cs = c_src = c).
__global__ void __launch_bounds__(kPrepThreads)
prepack_tc_kernel(const void* __restrict__ w, int wkind, int n, int taps, int c, int n_pad, int c_pad, int8_t* __restrict__ out,
                  int cs, int c_src)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kPrepThreads + threadIdx.x;
    const int64_t row_len = static_cast<int64_t>(taps) * c_pad;
    if (i >= n_pad * row_len) return;
    const int64_t row = i / row_len, rem = i - row * row_len;
    const int tap = static_cast<int>(rem / c_pad), ch = static_cast<int>(rem - static_cast<int64_t>(tap) * c_pad);
    int8_t v = 0;
    if (row < n && ch < c) {
        const int runs = c / cs, sub = ch / cs, cc = ch - sub * cs;
        if (cc < c_src)
            v = static_cast<int8_t>(qtz_dev::load_code_s8(w, wkind, row, (static_cast<int64_t>(tap) * runs + sub) * c_src + cc,
                                                static_cast<int64_t>(taps) * runs * c_src));
    }
    out[i] = v;
}

// int8 codes in [-8, 7] -> two per byte along the row (even element in the low nibble).
__global__ void __launch_bounds__(kPrepThreads)
pack_nibbles_kernel(const int8_t* __restrict__ w, int64_t bytes_out, uint8_t* __restrict__ out)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kPrepThreads + threadIdx.x;
    if (i >= bytes_out) return;
    out[i] = static_cast<uint8_t>((static_cast<uint32_t>(w[2 * i]) & 0xfu) | (static_cast<uint32_t>(w[2 * i + 1]) << 4));
}

// Weight sums per border class.  Class = 4 * rowclass + colclass, each a 2-bit mask
// (bit 0: first filter row/column is outside the image, bit 1: last one is).
__global__ void __launch_bounds__(kPrepThreads)
class_sums_kernel(const int8_t* __restrict__ wp, int n, int taps, int kw, int c_pad, int ncls, int32_t* __restrict__ wsum)
{
    __shared__ int32_t tapsum[9];
    const int row = blockIdx.x;
    if (threadIdx.x < 9) tapsum[threadIdx.x] = 0;
    __syncthreads();
    for (int tap = 0; tap < taps; ++tap) {
        int32_t s = 0;
        for (int ch = threadIdx.x; ch < c_pad; ch += kPrepThreads) s += wp[(static_cast<int64_t>(row) * taps + tap) * c_pad + ch];
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if ((threadIdx.x & 31) == 0 && s != 0) atomicAdd(&tapsum[tap], s);
    }
    __syncthreads();
    if (static_cast<int>(threadIdx.x) < ncls) {
        const int cls = threadIdx.x, rc = cls >> 2, cc = cls & 3;
        int32_t s = 0;
        if (taps == 1) {
            s = tapsum[0];
        } else {
            for (int i = 0; i < 3; ++i)
                for (int j = 0; j < kw; ++j) {
                    const bool cut = (i == 0 && (rc & 1)) || (i == 2 && (rc & 2)) || (j == 0 && (cc & 1)) || (j == 2 && (cc & 2));
                    if (!cut) s += tapsum[i * kw + j];
                }
        }
        wsum[static_cast<int64_t>(cls) * n + row] = s;
    }
}

// xsum[p] = sum of the c channel codes of input pixel p (for the -z_w sum(x) term).
__global__ void __launch_bounds__(kPrepThreads)
pixel_sum_kernel(const uint8_t* __restrict__ x, int64_t pixels, int c, int pitch, int32_t* __restrict__ xsum)
{
    // the convolution that follows needs these sums only in its epilogue: let it start now (its copies and MMAs run
    // beside this kernel; its epilogue waits for this grid before the first read of xsum)
    grid_launch_dependents();
    // this kernel itself may have started beside the tail of the kernel before it: its input may be that kernel's
    // output, and xsum may still be read by an earlier launch of the same plan
    grid_dependency_wait();
    const int warps_per_block = kPrepThreads / 32;
    const int lane = threadIdx.x & 31;
    for (int64_t p = static_cast<int64_t>(blockIdx.x) * warps_per_block + (threadIdx.x >> 5); p < pixels;
         p += static_cast<int64_t>(gridDim.x) * warps_per_block) {
        const uint8_t* row = x + p * pitch;
        uint32_t s = 0;
        auto take = [&](const uint4& v, int off) {
            const uint32_t words[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int first = off + 4 * i;
                uint32_t word = words[i];
                if (first + 4 > c) word = first >= c ? 0u : (word & (0xffffffffu >> (8 * (first + 4 - c))));
                s = __dp4a(word, 0x01010101u, s);
            }
        };
        int off = lane * 16;
        // four 16-byte loads of a lane in flight at a time (2 KB of the row per warp and step)
        for (; off + 3 * 512 < c; off += 4 * 512) {
            const uint4 v0 = __ldg(reinterpret_cast<const uint4*>(row + off));
            const uint4 v1 = __ldg(reinterpret_cast<const uint4*>(row + off + 512));
            const uint4 v2 = __ldg(reinterpret_cast<const uint4*>(row + off + 1024));
            const uint4 v3 = __ldg(reinterpret_cast<const uint4*>(row + off + 1536));
            take(v0, off); take(v1, off + 512); take(v2, off + 1024); take(v3, off + 1536);
        }
        for (; off < c; off += 512) take(__ldg(reinterpret_cast<const uint4*>(row + off)), off);
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) xsum[p] = static_cast<int32_t>(s);
    }
}

// Strided 1x1 convolution: copies the pixels the layer actually reads into a compact tensor.
__global__ void __launch_bounds__(kPrepThreads)
stride_gather_kernel(const uint8_t* __restrict__ x, uint8_t* __restrict__ out, int batch, int h, int w, int pitch,
                     int stride, int oh, int ow)
{
    grid_launch_dependents();      // the convolution launched next may set itself up beside this pre-pass (it waits for it before its first copy)
    const int chunks = pitch >> 4;
    const int64_t t = static_cast<int64_t>(blockIdx.x) * kPrepThreads + threadIdx.x;
    if (t >= static_cast<int64_t>(batch) * oh * ow * chunks) return;
    const int ck = static_cast<int>(t % chunks);
    int64_t p = t / chunks;
    const int ox = static_cast<int>(p % ow); p /= ow;
    const int oy = static_cast<int>(p % oh);
    const int64_t b = p / oh;
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(x + ((b * h + oy * stride) * w + ox * stride) * pitch) + ck);
    reinterpret_cast<uint4*>(out)[t] = v;
}

// Row-window layers (kw pixels of at most 16 channel bytes each: image stems).  The input is copied
// once into a frame of z_x codes (real zero, Section 2.1) with fp = 4, 8 or 16 bytes per pixel (the
// smallest that holds the channels and makes the step between output columns, stride * fp, a
// multiple of 16 bytes -- here exactly 16); rb / fp consecutive pixels of a frame row (rb = 32, 64
// or 128 bytes) are then one filter row of an output pixel's window plus zero-weight positions, and
// the window of the next output column starts 16 bytes later.  A tile (120 output columns of one
// output row) therefore needs, per filter row, one contiguous run of 16 * 119 + rb <= 2048 frame bytes
// in shared memory, and the tensor cores read their K-major operand rows straight out of that run
// through an unswizzled descriptor with a 16-byte row pitch (make_sliding_desc): no window matrix is
// ever materialised.  No border classes: padding is data.  One thread writes 16 bytes of the frame.
__global__ void __launch_bounds__(kPrepThreads)
pad_copy_kernel(const uint8_t* __restrict__ x, uint8_t* __restrict__ xp, int batch, int h, int w, int c, int hp, int wp,
                int pad, int zx, int fp, int in_words)
{
    grid_launch_dependents();      // the convolution launched next may set itself up beside this pre-pass (it waits for it before its first copy)
    const int ppc = 16 / fp;                         // pixels per 16-byte chunk
    const int chunks = wp / ppc;                     // wp is a multiple of ppc
    const int xc = blockIdx.x * blockDim.x + threadIdx.x;      // grid: (chunks of a row, frame rows, images)
    if (xc >= chunks) return;
    const int yp = blockIdx.y;
    const int64_t b = blockIdx.z;
    const int64_t i = (b * hp + yp) * chunks + xc;
    const int iy = yp - pad;
    const uint32_t zx4 = 0x01010101u * static_cast<uint32_t>(zx);
    uint32_t words[4] = {zx4, zx4, zx4, zx4};
    const int wpp = fp >> 2;                         // words per frame pixel
    if (iy >= 0 && iy < h) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {                // word k of the chunk: pixel k / wpp, channel word k % wpp
            const int j = k / wpp, q = k - j * wpp;
            const int ix = xc * ppc + j - pad;
            const int live = c - 4 * q;              // real channel bytes in this word
            if (ix < 0 || ix >= w || live <= 0) continue;
            uint32_t v = __ldg(reinterpret_cast<const uint32_t*>(x) + ((b * h + iy) * w + ix) * in_words + q);   // input pitch: 4 in_words bytes
            if (live < 4) {
                const uint32_t keep = 0xffffffffu >> (8 * (4 - live));
                v = (v & keep) | (zx4 & ~keep);
            }
            words[k] = v;
        }
    }
    reinterpret_cast<uint4*>(xp)[i] = make_uint4(words[0], words[1], words[2], words[3]);
}

// OHWI codes -> int8 [n_pad][taps][rb / fp pixels][fp bytes]: filter row dy of output channel `row` laid
// over the rb-byte run of frame pixels it meets; positions beyond kw pixels or c channels weigh zero.
// With several output rows per tile (bn_row < n_pad) matrix row j is channel j % bn_row of output row j / bn_row of
// the tile, and frame row f of the tile meets it with filter row f - (j / bn_row) * stride (zero outside 0 .. kh-1).
__global__ void __launch_bounds__(kPrepThreads)
prepack_rowwin_kernel(const void* __restrict__ w, int wkind, int n, int kh, int kw, int c, int n_pad, int fp, int rb,
                      int taps, int bn_row, int stride, int8_t* __restrict__ out)
{
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kPrepThreads + threadIdx.x;
    if (i >= static_cast<int64_t>(n_pad) * taps * rb) return;
    const int byte = static_cast<int>(i % rb);
    const int f = static_cast<int>((i / rb) % taps);
    const int64_t j = (i / rb) / taps;
    const int64_t row = j % bn_row;
    const int dy = f - static_cast<int>(j / bn_row) * stride;
    const int px = byte / fp, ch = byte % fp;
    int8_t v = 0;
    if (row < n && dy >= 0 && dy < kh && px < kw && ch < c)
        v = static_cast<int8_t>(qtz_dev::load_code_s8(w, wkind, row, (static_cast<int64_t>(dy) * kw + px) * c + ch, static_cast<int64_t>(kh) * kw * c));
    out[i] = v;
}

// Explicit im2col for layers with a short reduction (3-channel stem convolutions, strided 3x3):
// row p of `out` holds the window of output pixel p, filter rows first, then filter columns, then
// `cs` bytes per tap: the c channels and, where c is not a multiple of 4, padding bytes up to
// cs = roundup4(c) (the weights of the padding positions are zero).  Out-of-image taps and the
// padding bytes hold the code z_x (real zero, Section 2.1); the tail of the row up to its pitch is 0.
// The layer then runs as a pointwise layer over this matrix on the tensor cores.
//
// One CTA makes the rows of `tp` consecutive output pixels of one output row.  It first copies the
// kh input rows it needs into shared memory, cs bytes per pixel; a window is then kh contiguous runs
// of kw*cs bytes there, and every 32-bit word of an output row is one aligned word of shared memory.
// The CTA writes its rows with fully coalesced 16-byte stores.
__global__ void __launch_bounds__(kPrepThreads)
im2col_kernel(const uint8_t* __restrict__ x, uint8_t* __restrict__ out, int h, int w, int c, int cs, int pitch, int kh,
              int kw, int stride, int pad, int oh, int ow, int tp, int k_total, int k_pitch, int zx)
{
    grid_launch_dependents();      // the convolution launched next may set itself up beside this pre-pass (it waits for it before its first copy)
    extern __shared__ __align__(16) uint8_t im_s[];
    const int kwords = k_pitch >> 2;
    uint16_t* const off_s = reinterpret_cast<uint16_t*>(im_s);          // [kwords] word offset of output word k in the staged rows
    uint32_t* const rows_s = reinterpret_cast<uint32_t*>(im_s + ((2 * kwords + 15) & ~15));   // [kh][wt][cs / 4]
    const int wq = cs >> 2;                                              // words per pixel
    const int wt = (tp - 1) * stride + kw;                               // input pixels per staged row
    const int seg_w = (ow + tp - 1) / tp;
    int blk = blockIdx.x;
    const int seg = blk % seg_w; blk /= seg_w;
    const int oy = blk % oh;
    const int64_t b = blk / oh;
    const int ox0 = seg * tp;
    const int npx = min(tp, ow - ox0);
    const int iy0 = oy * stride - pad, ix0 = ox0 * stride - pad;
    const uint32_t zx4 = 0x01010101u * static_cast<uint32_t>(zx);

    const int run = kw * wq;                                             // words of one filter row
    for (int k = threadIdx.x; k < kwords; k += kPrepThreads) {
        const int dy = k / run;
        off_s[k] = static_cast<uint16_t>(4 * k < k_total ? dy * wt * wq + (k - dy * run) : 0);
    }
    // stage the input rows: one thread per word
    const uint8_t* const img = x + b * h * w * pitch;
    const int row_words = wt * wq;
    for (int dy = 0; dy < kh; ++dy) {
        const int iy = iy0 + dy;
        const bool row_in = iy >= 0 && iy < h;
        for (int e = threadIdx.x; e < row_words; e += kPrepThreads) {
            const int px = wq == 1 ? e : e / wq, q = e - px * wq;
            const int ix = ix0 + px;
            uint32_t v = zx4;
            if (row_in && ix >= 0 && ix < w) {
                v = __ldg(reinterpret_cast<const uint32_t*>(img + (static_cast<int64_t>(iy) * w + ix) * pitch) + q);
                const int live = c - 4 * q;                              // real channel bytes in this word
                if (live < 4) {
                    const uint32_t keep = 0xffffffffu >> (8 * (4 - live));
                    v = (v & keep) | (zx4 & ~keep);
                }
            }
            rows_s[dy * row_words + e] = v;
        }
    }
    __syncthreads();

    const int chunks = k_pitch >> 4;
    const int64_t row0 = (b * oh + oy) * ow + ox0;
    uint4* const dst = reinterpret_cast<uint4*>(out + row0 * k_pitch);
    const int tail_words = (k_total >> 2);                               // words at and beyond this index are zero
    int ck = threadIdx.x % chunks, p = threadIdx.x / chunks;
    const int step_p = kPrepThreads / chunks, step_ck = kPrepThreads - step_p * chunks;
    for (int i = threadIdx.x; i < npx * chunks; i += kPrepThreads) {
        const uint32_t* const win = rows_s + p * stride * wq;
        const uint2 o = *reinterpret_cast<const uint2*>(off_s + 4 * ck);
        uint32_t w0 = win[o.x & 0xffffu], w1 = win[o.x >> 16], w2 = win[o.y & 0xffffu], w3 = win[o.y >> 16];
        if (4 * ck + 4 > tail_words) {                                   // the row's last chunk: zero tail
            if (4 * ck + 0 >= tail_words) w0 = 0;
            if (4 * ck + 1 >= tail_words) w1 = 0;
            if (4 * ck + 2 >= tail_words) w2 = 0;
            if (4 * ck + 3 >= tail_words) w3 = 0;
        }
        dst[i] = make_uint4(w0, w1, w2, w3);
        p += step_p;
        ck += step_ck;
        if (ck >= chunks) {
            ck -= chunks;
            ++p;
        }
    }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
struct qtz_tc_state {
    TcArgs args{};
    qtz_conv_desc eff{};       // the layer as the kernel sees it (im2col layers become pointwise over the window matrix)
    bool im2col = false;
    bool strided_view = false; // strided 1x1 layer read through a strided tensor map (no gather pre-pass)
    bool rowwin = false;       // row-window layer: padded frame read through a sliding operand descriptor (see pad_copy_kernel)
    int hp = 0, wp = 0;        // its frame extent
    int fp = 16, rb = 128;     // bytes per frame pixel, bytes of one filter-row run
    size_t frame_bytes = 0;    // the frame with its slack
    int cs = 0;                // im2col: bytes per tap in the window matrix (channels rounded up to 4)
    CUtensorMap map_b{};
    CUtensorMap map_b_half{};  // pair mode: boxes of half the column tile
    bool pair = false;         // the layer runs on CTA pairs (clusters of two, tcgen05 cta_group::2)
    int pair_clusters = 0;     // pairs that can be resident at once
    int8_t* w_packed = nullptr;
    uint8_t* w_packed4 = nullptr;   // 4-bit layers: the same re-laid rows with two codes per byte (what the kernel reads when
                                    // the layer's weights are expanded in shared memory)
    int32_t* xsum = nullptr;
    int64_t in_pixels = 0;     // pixels of the (possibly gathered) input
    int in_h = 0, in_w = 0;    // its spatial extent
    int n_pad = 0;
    int swizzle_k = 0, swizzle_out = 0;
    uint32_t smem_bytes = 0;
    int grid = 0;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        (void)cudaGetLastError();
    }
    return fn;
}

CUtensorMapSwizzle swizzle_for(int bytes)
{
    switch (bytes) {
        case 128: return CU_TENSOR_MAP_SWIZZLE_128B;
        case 64: return CU_TENSOR_MAP_SWIZZLE_64B;
        case 32: return CU_TENSOR_MAP_SWIZZLE_32B;
        default: return CU_TENSOR_MAP_SWIZZLE_NONE;
    }
}

bool encode_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box, int swizzle_bytes)
{
    return qtz_encode_u8_map(m, base, rank, dims, strides_bytes, box, swizzle_bytes);
}

// The padded frame as a matrix of 8-byte elements, one row per frame row; a box is 2048 bytes of each of
// `rows` consecutive frame rows.
bool encode_frame_map(CUtensorMap* m, const void* base, int64_t row_bytes, int64_t frame_rows, int rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gd[2] = {static_cast<cuuint64_t>(row_bytes / 8), static_cast<cuuint64_t>(frame_rows)};
    cuuint64_t gs[1] = {static_cast<cuuint64_t>(row_bytes)};
    cuuint32_t bx[2] = {static_cast<cuuint32_t>(kRunBytes / 8), static_cast<cuuint32_t>(rows)};
    cuuint32_t es[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<void*>(base), gd, gs, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool is_pointwise(const qtz_conv_desc& d) { return d.kh == 1 && d.kw == 1 && d.pad == 0; }
bool is_3x3(const qtz_conv_desc& d) { return d.kh == 3 && d.kw == 3 && d.pad == 1 && d.stride == 1; }

// Row-window layers: see pad_copy_kernel.  Symmetric weights only (a zero-weight position must also
// be a zero in the integer arithmetic).  Frame pixel size: the smallest of 4, 8, 16 bytes that holds
// the channels and makes stride * fp exactly 16 (the row pitch of the sliding operand descriptor).
int rowwin_pixel_bytes(const qtz_conv_desc& d)
{
    for (int fp = 4; fp <= 16; fp *= 2)
        if (fp >= d.c && d.stride * fp == 16) return fp;
    return 0;
}

int rowwin_run_bytes(const qtz_conv_desc& d)
{
    const int fp = rowwin_pixel_bytes(d);
    if (fp == 0) return 0;
    for (int rb = 32; rb <= 128; rb *= 2)
        if (rb >= d.kw * fp) return rb;
    return 0;
}

bool wants_rowwin(const qtz_conv_desc& d, int w_zp_signed)
{
    if (is_pointwise(d) || (is_3x3(d) && d.c >= 8)) return false;
    return (d.c_pitch_in == 16 || d.c_pitch_in == 8 || d.c_pitch_in == 4) && rowwin_run_bytes(d) != 0 && d.kh <= 16 &&
           d.stride <= 4 && w_zp_signed == 0;
}

}  // namespace

bool qtz_encode_u8_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                       const uint32_t* box, int swizzle_bytes)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gd[4], gs[3];
    cuuint32_t bx[4], es[4];
    for (int i = 0; i < rank; ++i) {
        gd[i] = dims[i];
        bx[i] = box[i];
        es[i] = 1;
        if (i > 0) gs[i - 1] = strides_bytes[i - 1];
    }
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, static_cast<cuuint32_t>(rank), const_cast<void*>(base), gd, gs, bx, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_for(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Layers with a short reduction that are neither pointwise nor 3x3/stride 1 go through an explicit
// im2col and then run as pointwise layers.
static bool wants_im2col(const qtz_conv_desc& d)
{
    if (is_pointwise(d) || (is_3x3(d) && d.c >= 8)) return false;
    return static_cast<int64_t>(d.kh) * d.kw * d.c <= 1024 && d.kh <= 16 && d.kw <= 16;
}

bool qtz_tc_supported(const qtz_conv_desc& d)
{
    if (wants_im2col(d)) return true;
    if (!(is_pointwise(d) || is_3x3(d))) return false;
    if (is_pointwise(d) && d.stride > 4) return false;
    return true;
}

void qtz_tc_release(qtz_plan* p)
{
    if (!p->tc) return;
    cudaFree(p->tc->w_packed);
    cudaFree(p->tc->w_packed4);
    cudaFree(p->tc->xsum);
    delete p->tc;
    p->tc = nullptr;
}

qtz_status qtz_tc_prepare(qtz_plan* p, const void* w_q_dev, cudaStream_t st)
{
    qtz_ctx* h = p->h;
    if (!encode_fn()) {
        h->last_error = "cuTensorMapEncodeTiled is not available from the driver";
        return QTZ_ERR_CUDA;
    }
    qtz_tc_state* t = new (std::nothrow) qtz_tc_state();
    if (!t) return QTZ_ERR_INVALID_ARG;
    p->tc = t;
    t->eff = p->d;
    t->rowwin = wants_rowwin(p->d, p->w_zp_signed);
    t->im2col = !t->rowwin && wants_im2col(p->d);
    if ((p->d.c_pitch_in & 15) && !t->rowwin && !t->im2col) return QTZ_ERR_MISALIGNED;   // only the repacking paths take narrow pixels
    if (t->im2col) {
        const qtz_conv_desc& o = p->d;
        t->cs = (o.c + 3) / 4 * 4;
        const int k_total = o.kh * o.kw * t->cs;
        t->eff.h = p->oh; t->eff.w = p->ow;
        t->eff.c = k_total; t->eff.c_pitch_in = (k_total + 15) / 16 * 16;
        t->eff.kh = t->eff.kw = 1; t->eff.stride = 1; t->eff.pad = 0;
    }
    const qtz_conv_desc& d = t->eff;
    TcArgs& a = t->args;
    const bool pw = is_pointwise(d);
    const bool rw = t->rowwin;
    a.taps = rw ? d.kh : (pw ? 1 : 9);       // row-window layers: one "tap" per filter row
    a.kw = (pw || rw) ? 1 : 3;
    a.pad = (pw || rw) ? 0 : 1;
    a.cstride = rw ? d.stride : 0;
    if (rw) {
        t->fp = rowwin_pixel_bytes(d);
        t->rb = rowwin_run_bytes(d);
        const int ppc = 16 / t->fp;               // frame rows are whole 16-byte chunks
        t->hp = (d.h + 2 * d.pad + d.stride - 1) / d.stride * d.stride;
        t->wp = (std::max(d.w + 2 * d.pad, (p->ow - 1) * d.stride + t->rb / t->fp) + ppc - 1) / ppc * ppc;
    }
    a.N = d.n;
    a.B = d.batch;
    a.H = p->oh;
    a.W = p->ow;
    t->in_h = p->oh;  // after the optional stride gather the input has the output's extent
    t->in_w = p->ow;
    t->in_pixels = static_cast<int64_t>(d.batch) * p->oh * p->ow;

    // K blocking: the widest swizzle the channel count fills reasonably
    a.BK = rw ? t->rb : (d.c > 64 ? 128 : (d.c > 32 ? 64 : 32));
    a.c_pad = rw ? t->rb : (d.c + a.BK - 1) / a.BK * a.BK;
    a.kb_per_tap = a.c_pad / a.BK;
    // N tiling: as few tiles as possible, each a multiple of 32 columns
    a.n_tiles = (d.n + 255) / 256;
    {   // a layer with few pixel tiles (a classifier: one or two) spreads over the SMs by its columns instead
        const int64_t m_tiles = (t->in_pixels + kTileM - 1) / kTileM;
        if (pw && d.n > 64 && m_tiles * a.n_tiles * 2 <= h->num_sms)
            a.n_tiles = static_cast<int32_t>(std::max<int64_t>(a.n_tiles, std::min<int64_t>((d.n + 63) / 64, h->num_sms / m_tiles)));
    }
    // (one tile: 32-column granularity, the TMA store clips what lies beyond the real channels;
    //  several tiles: whole staging boxes, since a box must not spill into the next tile's columns)
    a.BN = a.n_tiles == 1 ? (d.n + 31) / 32 * 32 : ((d.n + a.n_tiles - 1) / a.n_tiles + 63) / 64 * 64;
    a.n_tiles = (d.n + a.BN - 1) / a.BN;     // rounding the width up may have emptied the last tile
    // (a single column tile wider than 128 also takes 128-byte boxes: the store clips the last one at N, and every
    //  box row is one request to the copy engine whatever its length)
    a.out_box = (a.BN % 128 == 0 || (a.n_tiles == 1 && a.BN > 128)) ? 128 : 64;
    // every accumulator a tile ahead lets the MMA warp start a tile before an epilogue group is back
    a.n_acc = std::min(kMaxAcc, kTmemCols / a.BN);
    a.acc_stride = a.BN;
    // Row-window layers with few output channels: several output rows per tile (see TcArgs::rrows).  As many rows (4 or
    // 2) as keep the tile within 256 columns and the widened weights resident in shared memory.
    a.rrows = 1;
    a.bn_row = a.BN;
    if (rw && a.n_tiles == 1 && d.outkind == QTZ_OUT_U8 && (a.BN == 32 || a.BN == 64 || a.BN == 128) && !h->single_row_stems) {
        for (int r = 4; r >= 2; r >>= 1) {
            const int taps_r = (r - 1) * d.stride + d.kh;
            if (r * a.BN <= 256 && r <= p->oh && static_cast<int64_t>(taps_r) * r * a.BN * t->rb <= kResidentBMax) {
                a.rrows = r;
                break;
            }
        }
        if (a.rrows > 1) {
            a.out_box = a.BN;                                 // one staging box per output row
            a.BN *= a.rrows;
            a.taps = (a.rrows - 1) * d.stride + d.kh;          // frame rows a tile reads
            a.n_acc = std::min(kMaxAcc, kTmemCols / a.BN);
            a.acc_stride = a.BN;
            // the frame reaches down to the last frame row of the last tile
            const int tiles_h = (p->oh + a.rrows - 1) / a.rrows;
            t->hp = std::max(t->hp, ((tiles_h * a.rrows - 1) * d.stride + d.kh + d.stride - 1) / d.stride * d.stride);
        }
    }
    t->n_pad = a.n_tiles * a.BN;
    a.ncls = (pw || rw) ? 1 : kMaxCls;

    // pixel tiling
    // (a strided 1x1 layer with symmetric weights reads its input through a strided view of the tensor -- every
    //  stride-th pixel of every stride-th row -- and is tiled as boxes of that view; with a weight zero point the
    //  activation sums need the compacted copy, so those layers gather first)
    const bool strided_view = pw && d.stride > 1 && p->w_zp_signed == 0;
    t->strided_view = strided_view;
    if (pw && !strided_view) {
        a.is4d = 0;
        a.tw = kTileM; a.th = 1; a.tb = 1; a.rows = kTileM;
        a.tiles_w = static_cast<int32_t>((t->in_pixels + kTileM - 1) / kTileM);
        a.tiles_h = 1;
        if (static_cast<int64_t>(a.tiles_w) * a.n_tiles > 0x7fffffff) return QTZ_ERR_UNSUPPORTED;
        a.num_tiles = static_cast<uint32_t>(a.tiles_w) * a.n_tiles;
        // the 2-D view treats all pixels as one row of length M
        a.W = static_cast<int32_t>(t->in_pixels);
        a.H = 1;
        a.B = 1;
        if (t->in_pixels > 0x7fffffff) return QTZ_ERR_UNSUPPORTED;
    } else {
        a.is4d = 1;
        int64_t best_tiles = INT64_MAX;
        if (rw) {
            // a tile is a run of 128 output columns of one output row (columns beyond the image are
            // computed from whatever follows in the frame and clipped by the store)
            a.tw = kRunCols; a.th = 1; a.tb = 1;
            best_tiles = static_cast<int64_t>((a.W + kRunCols - 1) / kRunCols) * ((a.H + a.rrows - 1) / a.rrows) * a.B;
        } else {
            for (int tw = 1; tw <= std::min(a.W, kTileM); ++tw)
                for (int th = 1; th <= std::min(a.H, kTileM / tw); ++th) {
                    const int tb = std::min(a.B, kTileM / (tw * th));
                    const int64_t tiles = static_cast<int64_t>((a.W + tw - 1) / tw) * ((a.H + th - 1) / th) * ((a.B + tb - 1) / tb);
                    if (tiles < best_tiles || (tiles == best_tiles && tw > a.tw)) {
                        best_tiles = tiles;
                        a.tw = tw; a.th = th; a.tb = tb;
                    }
                }
        }
        a.rows = a.tw * a.th * a.tb;
        a.tiles_w = (a.W + a.tw - 1) / a.tw;
        a.tiles_h = (a.H + a.th * a.rrows - 1) / (a.th * a.rrows);
        if (best_tiles * a.n_tiles > 0x7fffffff) return QTZ_ERR_UNSUPPORTED;
        a.num_tiles = static_cast<uint32_t>(best_tiles * a.n_tiles);
    }
    for (int cls = 0; cls < kMaxCls; ++cls) {
        const int rc = cls >> 2, cc = cls & 3;
        const int rows_valid = pw ? 1 : 3 - (rc & 1) - ((rc >> 1) & 1);
        const int cols_valid = pw ? 1 : 3 - (cc & 1) - ((cc >> 1) & 1);
        a.kvalid[cls] = rows_valid * cols_valid * d.c;
    }

    a.m_tiles = static_cast<int32_t>(a.num_tiles / a.n_tiles);
    // CTA pairs for GEMM-like pointwise layers: full-width column tiles, a reduction and a width of at least 2048 and
    // at least two tiles per SM.  A pair works on 256 pixels x 256 columns, each CTA fetching half of every weight K block.
    a.pair = 0;
    // (measured: layers of the networks with K = 1024..2048 and a few hundred tiles, which are bound by HBM and by
    //  latency rather than by the tensor cores, run about 10 % slower on pairs, so the bar is set above them)
    if (pw && !strided_view && a.BN == 256 && d.c >= 2048 && d.n >= 2048 && a.num_tiles >= 2 * static_cast<uint32_t>(h->num_sms) && !h->no_pairs) {
        int clusters = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(h->num_sms / 2 * 2));
        cfg.blockDim = dim3(kThreadsTc);
        cfg.dynamicSmemBytes = 227 * 1024;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension;
        at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        (void)cudaFuncSetAttribute(conv_tc_kernel<true, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (cudaOccupancyMaxActiveClusters(&clusters, conv_tc_kernel<true, 0>, &cfg) == cudaSuccess && clusters >= h->num_sms / 4) {
            a.pair = 1;
            t->pair = true;
            a.m_tiles = (a.m_tiles + 1) / 2;
            a.num_tiles = static_cast<uint32_t>(a.m_tiles) * a.n_tiles;
            t->pair_clusters = clusters;
        }
        (void)cudaGetLastError();
    }
    a.group_m = std::max(1, std::min(a.m_tiles, 16));
    a.dv_per_group = make_fastdiv(static_cast<uint32_t>(a.group_m) * a.n_tiles);
    a.dv_group_m = make_fastdiv(static_cast<uint32_t>(a.group_m));
    a.dv_group_last = make_fastdiv(static_cast<uint32_t>(std::max(1, a.m_tiles % a.group_m)));
    a.dv_tiles_w = make_fastdiv(static_cast<uint32_t>(a.tiles_w));
    a.dv_tiles_h = make_fastdiv(static_cast<uint32_t>(std::max(1, a.tiles_h)));
    // shared-memory budget -> pipeline depth
    // worst case (all border classes) for the smem opt-in; every launch picks its own depth
    a.groups = 1;
    a.gwarps = 8;
    a.obuf = 1;
    a.bres = 0;
    a.spb = 1;
    a.stages = 2;
    if (make_layout(a.BK, a.BN, 2, a.ncls, a.out_box, 1, 1, 0, 1).total > static_cast<uint32_t>(kSmemBudget)) return QTZ_ERR_UNSUPPORTED;

    // instruction descriptor: s32 accumulate, A = u8, B = s8, both K-major, N and M of the tile
    a.idesc = (2u << 4) | (0u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) |
              (static_cast<uint32_t>((a.pair ? 2 * kTileM : kTileM) >> 4) << 24);

    // weights: re-lay, then the per-class sums
    const int64_t wbytes = static_cast<int64_t>(t->n_pad) * a.taps * a.c_pad;
    QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&t->w_packed), static_cast<size_t>(wbytes)));
    if (rw)
        prepack_rowwin_kernel<<<static_cast<unsigned>((wbytes + kPrepThreads - 1) / kPrepThreads), kPrepThreads, 0, st>>>(
            w_q_dev, d.wkind, d.n, d.kh, d.kw, d.c, t->n_pad, t->fp, t->rb, a.taps, a.rrows > 1 ? a.bn_row : t->n_pad, d.stride, t->w_packed);
    else
        prepack_tc_kernel<<<static_cast<unsigned>((wbytes + kPrepThreads - 1) / kPrepThreads), kPrepThreads, 0, st>>>(
            w_q_dev, d.wkind, d.n, a.taps, d.c, t->n_pad, a.c_pad, t->w_packed, t->im2col ? t->cs : d.c, t->im2col ? p->d.c : d.c);
    QTZ_LAUNCH_CHECK(h, "prepack_tc_kernel");
    if (d.wkind == QTZ_W_S4_PACKED_PER_CHANNEL_SYM) {
        QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&t->w_packed4), static_cast<size_t>(wbytes / 2)));
        pack_nibbles_kernel<<<static_cast<unsigned>((wbytes / 2 + kPrepThreads - 1) / kPrepThreads), kPrepThreads, 0, st>>>(
            t->w_packed, wbytes / 2, t->w_packed4);
        QTZ_LAUNCH_CHECK(h, "pack_nibbles_kernel");
    }
    QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&p->wsum), sizeof(int32_t) * a.ncls * d.n));
    if (rw)   // one class, the whole packed row as a single run
        class_sums_kernel<<<d.n, kPrepThreads, 0, st>>>(t->w_packed, d.n, 1, 1, a.taps * a.c_pad, 1, p->wsum);
    else
        class_sums_kernel<<<d.n, kPrepThreads, 0, st>>>(t->w_packed, d.n, a.taps, a.kw, a.c_pad, a.ncls, p->wsum);
    QTZ_LAUNCH_CHECK(h, "class_sums_kernel");

    if (p->w_zp_signed != 0)
        QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&t->xsum), sizeof(int32_t) * static_cast<size_t>(t->in_pixels)));
    if ((pw && d.stride > 1 && !strided_view) || t->im2col)
        QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&p->x_gather), static_cast<size_t>(t->in_pixels) * d.c_pitch_in));
    if (rw) {
        // the last tiles of a row read past its end (into the next row, or into this slack after the last one)
        a.frame_row = static_cast<int64_t>(t->wp) * t->fp;
        a.frame_rows = t->hp;
        // a copy brings 2048 bytes of each filter row (the row's end and whatever lies past the image arrive as
        // zeros); the MMA reads 16 * 127 + rb bytes per row, i.e. up to 112 bytes into the next row's slot, which only
        // accumulator rows beyond the 120 columns of a tile ever see
        a.seg_bytes = kRunBytes;
        a.a_blk = kRunBytes;
        const size_t slack = static_cast<size_t>(a.tiles_w) * kTileM * 16 + 256;
        t->frame_bytes = static_cast<size_t>(d.batch) * t->hp * a.frame_row + slack;
        if (t->frame_bytes / 8 > 0x7fffffffull) return QTZ_ERR_UNSUPPORTED;      // element indices are 32-bit
        QTZ_CUDA(h, cudaMalloc(reinterpret_cast<void**>(&p->x_gather), t->frame_bytes));
        QTZ_CUDA(h, cudaMemsetAsync(p->x_gather, 0, t->frame_bytes, st));
    }

    // the weight map never changes
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(a.taps) * a.c_pad, static_cast<uint64_t>(t->n_pad)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.taps) * a.c_pad};
        const uint32_t box[2] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(a.BN)};
        if (!encode_map(&t->map_b, t->w_packed, 2, dims, strides, box, a.BK)) {
            h->last_error = "cuTensorMapEncodeTiled failed for the weight tensor";
            return QTZ_ERR_CUDA;
        }
        const uint32_t half_box[2] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(a.BN / 2)};
        if (t->pair && !encode_map(&t->map_b_half, t->w_packed, 2, dims, strides, half_box, a.BK)) {
            h->last_error = "cuTensorMapEncodeTiled failed for the weight tensor (half tiles)";
            return QTZ_ERR_CUDA;
        }
    }
    a.bias = p->bias;
    a.wsum = p->wsum;
    a.mult = p->mult;
    a.rshift = p->rshift;
    a.xsum = t->xsum;
    a.zw = p->w_zp_signed;
    a.raw = d.outkind == QTZ_OUT_S32_RAW;
    a.fast_requant = (!a.raw && p->rshift_min >= 33 && p->rshift_max <= 53) ? 1 : 0;
    a.fold = 0;                             // decided per launch (it depends on the zero points)
    a.status = h->status_dev;
    a.wait_budget = h->wait_budget;
    t->grid = t->pair ? 2 * static_cast<int>(std::min<int64_t>(a.num_tiles, t->pair_clusters))
                      : static_cast<int>(std::min<int64_t>(a.num_tiles, h->num_sms));

    // per device, so set for the device of this plan every time (the call is cheap)
    QTZ_CUDA(h, cudaFuncSetAttribute(conv_tc_kernel<false, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
    return QTZ_OK;
}

qtz_status qtz_tc_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, void* y, int32_t y_zp, int32_t act_min,
                         int32_t act_max, cudaStream_t st, const qtz_residual* res, const uint8_t* s_dev)
{
    qtz_ctx* h = p->h;
    qtz_tc_state* t = p->tc;
    const qtz_conv_desc& d = t->eff;
    TcArgs a = t->args;
    a.wait_budget = h->wait_budget;
    const bool pw = is_pointwise(d);

    const uint8_t* xin = x;
    if (t->rowwin) {
        const int chunks = t->wp * t->fp / 16;
        if (t->hp > 65535 || d.batch > 65535) return QTZ_ERR_UNSUPPORTED;
        const int threads = std::min(kPrepThreads, (chunks + 31) / 32 * 32);
        pad_copy_kernel<<<dim3(static_cast<unsigned>((chunks + threads - 1) / threads), static_cast<unsigned>(t->hp),
                               static_cast<unsigned>(d.batch)), threads, 0, st>>>(
            x, p->x_gather, d.batch, d.h, d.w, d.c, t->hp, t->wp, d.pad, x_zp, t->fp, d.c_pitch_in / 4);
        QTZ_LAUNCH_CHECK(h, "pad_copy_kernel");
        xin = p->x_gather;
    } else if (t->im2col) {
        const qtz_conv_desc& o = p->d;
        // pixels per CTA: as many as keep the staged input rows within 40 KB
        int tp = 64;
        while (tp > 8 && static_cast<int64_t>(o.kh) * ((tp - 1) * o.stride + o.kw) * t->cs > 40 * 1024) tp >>= 1;
        const size_t smem = ((static_cast<size_t>(d.c_pitch_in) / 2 + 15) & ~static_cast<size_t>(15)) +
                            static_cast<size_t>(o.kh) * ((tp - 1) * o.stride + o.kw) * t->cs;
        const int64_t blocks = static_cast<int64_t>(o.batch) * p->oh * ((p->ow + tp - 1) / tp);
        im2col_kernel<<<static_cast<unsigned>(blocks), kPrepThreads, smem, st>>>(
            x, p->x_gather, o.h, o.w, o.c, t->cs, o.c_pitch_in, o.kh, o.kw, o.stride, o.pad, p->oh, p->ow, tp, d.c, d.c_pitch_in, x_zp);
        QTZ_LAUNCH_CHECK(h, "im2col_kernel");
        xin = p->x_gather;
    } else if (pw && d.stride > 1 && !t->strided_view) {
        const int64_t work = t->in_pixels * (d.c_pitch_in >> 4);
        stride_gather_kernel<<<static_cast<unsigned>((work + kPrepThreads - 1) / kPrepThreads), kPrepThreads, 0, st>>>(
            x, p->x_gather, d.batch, d.h, d.w, d.c_pitch_in, d.stride, p->oh, p->ow);
        QTZ_LAUNCH_CHECK(h, "stride_gather_kernel");
        xin = p->x_gather;
    }
    if (a.zw != 0) {
        // the convolution starts beside this pre-pass (programmatic dependent launch), so the profiling events
        // bracket the two together
        if (p->ev_start) QTZ_CUDA(h, cudaEventRecord(p->ev_start, st));
        const int blocks = static_cast<int>(std::min<int64_t>((t->in_pixels + 7) / 8, static_cast<int64_t>(h->num_sms) * 16));
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(blocks));
        cfg.blockDim = dim3(kPrepThreads);
        cfg.stream = st;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        QTZ_CUDA(h, cudaLaunchKernelEx(&cfg, pixel_sum_kernel, xin, t->in_pixels, static_cast<int>(d.c), static_cast<int>(d.c_pitch_in), t->xsum));
        QTZ_LAUNCH_CHECK(h, "pixel_sum_kernel");
    }

    if (res && a.raw) return QTZ_ERR_UNSUPPORTED;
    CUtensorMap map_a, map_y, map_s;
    const uint64_t pitch = static_cast<uint64_t>(d.c_pitch_in);
    if (t->rowwin) {
        map_a = t->map_b;   // encoded below, once the number of filter rows per ring stage is known
    } else if (t->strided_view) {
        // every stride-th pixel of every stride-th row, as a tensor of the output's extent
        const uint64_t sv = static_cast<uint64_t>(p->d.stride);
        const uint64_t dims[4] = {static_cast<uint64_t>(d.c), static_cast<uint64_t>(p->ow), static_cast<uint64_t>(p->oh),
                                  static_cast<uint64_t>(d.batch)};
        const uint64_t strides[3] = {pitch * sv, pitch * p->d.w * sv, pitch * p->d.w * p->d.h};
        const uint32_t box[4] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(a.tw), static_cast<uint32_t>(a.th),
                                 static_cast<uint32_t>(a.tb)};
        if (!encode_map(&map_a, xin, 4, dims, strides, box, a.BK)) return QTZ_ERR_CUDA;
    } else if (pw) {
        const uint64_t dims[2] = {static_cast<uint64_t>(d.c), static_cast<uint64_t>(t->in_pixels)};
        const uint64_t strides[1] = {pitch};
        const uint32_t box[2] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(kTileM)};
        if (!encode_map(&map_a, xin, 2, dims, strides, box, a.BK)) return QTZ_ERR_CUDA;
    } else {
        const uint64_t dims[4] = {static_cast<uint64_t>(d.c), static_cast<uint64_t>(d.w), static_cast<uint64_t>(d.h),
                                  static_cast<uint64_t>(d.batch)};
        const uint64_t strides[3] = {pitch, pitch * d.w, pitch * d.w * d.h};
        const uint32_t box[4] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(a.tw), static_cast<uint32_t>(a.th),
                                 static_cast<uint32_t>(a.tb)};
        if (!encode_map(&map_a, xin, 4, dims, strides, box, a.BK)) return QTZ_ERR_CUDA;
    }
    map_s = t->map_b;      // placeholder unless a residual add is fused
    if (a.raw) {
        map_y = t->map_b;  // unused by the kernel in this mode
        a.y_raw = static_cast<int32_t*>(y);
    } else {
        const uint64_t opitch = static_cast<uint64_t>(d.c_pitch_out);
        if (pw && !t->strided_view) {
            const uint64_t dims[2] = {static_cast<uint64_t>(d.n), static_cast<uint64_t>(t->in_pixels)};
            const uint64_t strides[1] = {opitch};
            const uint32_t box[2] = {static_cast<uint32_t>(a.out_box), static_cast<uint32_t>(kTileM)};
            if (!encode_map(&map_y, y, 2, dims, strides, box, a.out_box)) return QTZ_ERR_CUDA;
            if (res && !encode_map(&map_s, s_dev, 2, dims, strides, box, a.out_box)) return QTZ_ERR_CUDA;
        } else {
            const uint64_t dims[4] = {static_cast<uint64_t>(d.n), static_cast<uint64_t>(p->ow), static_cast<uint64_t>(p->oh),
                                      static_cast<uint64_t>(d.batch)};
            const uint64_t strides[3] = {opitch, opitch * p->ow, opitch * p->ow * p->oh};
            const uint32_t box[4] = {static_cast<uint32_t>(a.out_box), static_cast<uint32_t>(a.tw), static_cast<uint32_t>(a.th),
                                     static_cast<uint32_t>(a.tb)};
            if (!encode_map(&map_y, y, 4, dims, strides, box, a.out_box)) return QTZ_ERR_CUDA;
            if (res && !encode_map(&map_s, s_dev, 4, dims, strides, box, a.out_box)) return QTZ_ERR_CUDA;
        }
    }
    a.zx = x_zp;
    a.zy = y_zp;
    a.act_min = act_min;
    a.act_max = act_max;
    a.res = 0;
    if (res) {
        // the requantisation of the epilogue produces t with its own quantizer; the add then produces y
        a.res = 1;
        a.zy = res->t_zero_point;
        a.act_min = res->t_act_min;
        a.act_max = res->t_act_max;
        a.res_rule = qtz_add::AddRule{res->t_zero_point, res->t_mult, res->s_zero_point, res->s_mult, res->rshift, y_zp, act_min, act_max};
        a.res_kind = (res->rshift >= 16 && res->rshift <= 38) ? 3 : (res->rshift >= 32 ? 0 : (res->rshift >= 10 ? 1 : 2));
        a.res_split = qtz_add::make_split(a.res_rule);
        a.res_addend = qtz_add::add_addend(a.res_rule);
    }
    // with z_x = 0 the cross-term correction no longer depends on the border class: one class, small tables
    if (x_zp == 0) a.ncls = 1;
    // Shared memory is split between the operand ring, the epilogue groups and their staging boxes.
    // Preference: many groups (overlapped tile drains) with two or three boxes each (the store of one box
    // overlaps the arithmetic of the next), as long as the ring keeps four stages, or the whole
    // reduction plus one block when that is shorter.  Four groups need four accumulators in TMEM.
    auto depth = [&](int groups, int obuf) {
        int st_ = kMaxStages;
        for (; st_ >= 2; --st_)
            if (make_layout(a.BK, a.BN, st_, a.ncls, a.out_box, groups, obuf, a.bres, a.spb, a.a_blk, a.pair).total <= static_cast<uint32_t>(kSmemBudget)) break;
        return st_;
    };
    const int kblocks = a.taps * a.kb_per_tap;
    // weights of a single-column-tile layer stay resident when they are small: the ring then carries activations only
    // (4-bit layers expand their packed codes in shared memory, which needs them resident: they get a larger share,
    //  and a layer with several column tiles qualifies when every CTA runs a single tile -- a classifier)
    const bool one_tile_each = a.num_tiles <= static_cast<uint32_t>(t->grid);
    if (t->w_packed4)
        a.bres = ((a.n_tiles == 1 || one_tile_each) && kblocks * a.BN * a.BK <= kResidentB4Max) ? kblocks : 0;
    else
        a.bres = (a.n_tiles == 1 && kblocks * a.BN * a.BK <= kResidentBMax) ? kblocks : 0;
    if (a.pair) a.bres = 0;                          // a pair streams its weight halves
    // several K blocks share a ring stage (one barrier handshake for all of them) while the stage stays within 32 KB
    auto blocks_per_stage = [&]() {
        const int blk = (a.a_blk > 0 ? a.a_blk : kTileM * a.BK) + (a.bres > 0 ? 0 : (a.pair ? a.BN / 2 : a.BN) * a.BK);
        int best = 1;
        for (int c = 2; c <= (a.a_blk > 0 ? 8 : 4); ++c)
            if (kblocks % c == 0 && c * blk <= 32 * 1024) best = c;
        return best;
    };
    a.spb = blocks_per_stage();
    int need = std::min(4, kblocks / a.spb + 1);
    if (a.pair) need = 6;                            // the pair's hand-offs cross SMs: a deeper ring, fewer staging boxes
    static const int choice[7][2] = {{4, 3}, {4, 2}, {2, 3}, {2, 2}, {1, 2}, {2, 1}, {1, 1}};
    // attempts: resident weights with several K blocks per stage; resident weights with one K block per stage (a
    // smaller ring beside a large resident tile); weights through the ring
    for (int attempt = 0; attempt < 3; ++attempt) {
        a.groups = 1;
        a.obuf = 1;
        bool found = false;
        for (const auto& c : choice) {
            if (c[0] == 4 && a.n_acc < 4) continue;
            const int ob = a.raw ? 1 : c[1];         // the boxes rotate across tiles as well
            if (depth(c[0], ob) >= need) {
                a.groups = c[0];
                a.obuf = ob;
                found = true;
                break;
            }
        }
        if (found || a.bres == 0) break;
        if (attempt == 0 && a.spb > 1) {
            a.spb = 1;
        } else {
            a.bres = 0;                              // no room beside resident weights: send them through the ring
            a.spb = blocks_per_stage();
        }
        need = std::min(4, kblocks / a.spb + 1);
    }
    a.gwarps = a.groups == 4 ? 4 : 8;
    a.stages = depth(a.groups, a.obuf);
    if (a.stages < 2) return QTZ_ERR_UNSUPPORTED;
    const uint32_t smem_bytes = make_layout(a.BK, a.BN, a.stages, a.ncls, a.out_box, a.groups, a.obuf, a.bres, a.spb, a.a_blk, a.pair).total + 1024;
    // folded form: shifts 32..53 (the high word of the 64-bit sum, shifted on by r - 32)
    // (2: shifts below 32 as well, given that no requantised value can leave 32 bits)
    a.fold = 0;
    if (!a.raw && a.ncls == 1 && a.zw == 0 && p->rshift_max <= 53)
        a.fold = p->rshift_min >= 32 ? 1 : (p->narrow_ok ? 2 : 0);
    if (t->rowwin && !encode_frame_map(&map_a, xin, a.frame_row, static_cast<int64_t>(d.batch) * t->hp, a.spb)) return QTZ_ERR_CUDA;
    // thread copies for the frame runs of row-window layers (see TcArgs::lsu).  (For pointwise tiles with short
    // rows one warp's 16-byte copies were slower than the copy engine: about 140 cycles per warp-wide copy.)
    a.lsu = (a.stages >= 3 && t->rowwin) ? 1 : 0;
    a.src = xin;
    a.full_count = a.lsu ? (a.bres > 0 ? 1 : 2) : 1;
    a.w4 = (t->w_packed4 && a.bres > 0) ? t->w_packed4 : nullptr;
    a.w4_row = (a.taps * a.c_pad) >> 1;
    p->detail = std::string("tcgen05") + (t->rowwin ? " row-window" : (t->im2col ? " im2col" : (pw ? (t->strided_view ? " pointwise strided-view" : " pointwise") : " 3x3"))) +
                (a.bres > 0 ? (a.w4 ? " weights:int4-expanded-in-smem" : " weights:resident") : " weights:streamed") +
                (a.pair ? " cta-pairs" : "") + (a.rrows > 1 ? " rows-per-tile:" + std::to_string(a.rrows) : std::string()) +
                (a.res ? " +residual-add" : "");
    if (p->ev_start && a.zw == 0) QTZ_CUDA(h, cudaEventRecord(p->ev_start, st));
    {
        // cluster of two for the pair form; early start beside pixel_sum_kernel when that kernel was just launched
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(t->grid));
        cfg.blockDim = dim3(kThreadsTc);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute at[2];
        unsigned n_at = 0;
        if (t->pair) {
            at[n_at].id = cudaLaunchAttributeClusterDimension;
            at[n_at].val.clusterDim.x = 2; at[n_at].val.clusterDim.y = 1; at[n_at].val.clusterDim.z = 1;
            ++n_at;
        }
        {   // early start beside the tail of the previous kernel (fully serial unless that kernel allows dependents)
            at[n_at].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            at[n_at].val.programmaticStreamSerializationAllowed = 1;
            ++n_at;
        }
        cfg.attrs = at;
        cfg.numAttrs = n_at;
        if (t->pair)
            QTZ_CUDA(h, cudaLaunchKernelEx(&cfg, conv_tc_kernel<true, 0>, map_a, t->map_b_half, map_y, map_s, a));
        else
            QTZ_CUDA(h, cudaLaunchKernelEx(&cfg, conv_tc_kernel<false, 0>, map_a, t->map_b, map_y, map_s, a));
    }
    QTZ_LAUNCH_CHECK(h, "conv_tc_kernel");
    if (p->ev_stop) QTZ_CUDA(h, cudaEventRecord(p->ev_stop, st));
    return QTZ_OK;
}

// Depthwise 3x3 -> pointwise in one kernel (see DwFront).  QTZ_ERR_UNSUPPORTED when this pair of layers cannot run
// that way; the caller then runs the two plans one after the other, with the same result.
qtz_status qtz_tc_launch_dw_pw(qtz_plan* dwp, qtz_plan* p, const uint8_t* x, int32_t x_zp, int32_t mid_zp, int32_t mid_min,
                               int32_t mid_max, void* y, int32_t y_zp, int32_t act_min, int32_t act_max, cudaStream_t st)
{
    qtz_ctx* h = p->h;
    qtz_tc_state* t = p->tc;
    const qtz_conv_desc& d = p->d;       // the pointwise layer
    const qtz_conv_desc& dd = dwp->d;    // the depthwise layer
    if (!t || t->rowwin || t->im2col || t->pair || t->w_packed4 || !is_pointwise(d) || d.stride != 1) return QTZ_ERR_UNSUPPORTED;
    if (d.outkind != QTZ_OUT_U8 || dd.outkind != QTZ_OUT_U8 || p->w_zp_signed != 0 || dwp->w_zp_signed != 0) return QTZ_ERR_UNSUPPORTED;
    if (dwp->rshift_min < 32 || dwp->rshift_max > 53 || (dd.stride != 1 && dd.stride != 2)) return QTZ_ERR_UNSUPPORTED;
    if (d.c != dd.c || d.batch != dd.batch || d.h != dwp->oh || d.w != dwp->ow || (dd.c & 3)) return QTZ_ERR_INVALID_ARG;
    TcArgs a = t->args;
    a.wait_budget = h->wait_budget;
    // one column tile over all output channels (several would each repeat the depthwise work of their pixels), whatever
    // split the plan chose for the pointwise layer alone
    if (d.n > 256) return QTZ_ERR_UNSUPPORTED;
    a.n_tiles = 1;
    a.BN = (d.n + 31) / 32 * 32;
    a.out_box = (a.BN % 128 == 0 || a.BN > 128) ? 128 : 64;
    a.n_acc = std::min(kMaxAcc, kTmemCols / a.BN);
    a.acc_stride = a.BN;
    a.idesc = (2u << 4) | (0u << 7) | (1u << 10) | (static_cast<uint32_t>(a.BN >> 3) << 17) | (static_cast<uint32_t>(kTileM >> 4) << 24);
    if (a.BN > t->n_pad) return QTZ_ERR_UNSUPPORTED;
    CUtensorMap map_b;
    {
        const uint64_t dims[2] = {static_cast<uint64_t>(a.taps) * a.c_pad, static_cast<uint64_t>(t->n_pad)};
        const uint64_t strides[1] = {static_cast<uint64_t>(a.taps) * a.c_pad};
        const uint32_t box[2] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(a.BN)};
        if (!encode_map(&map_b, t->w_packed, 2, dims, strides, box, a.BK)) return QTZ_ERR_CUDA;
    }
    const int kblocks = a.kb_per_tap;
    if (static_cast<int64_t>(kblocks) * a.BN * a.BK > kResidentBMax) return QTZ_ERR_UNSUPPORTED;
    a.bres = kblocks;
    a.spb = 1;
    a.is4d = 1;
    a.W = p->ow; a.H = p->oh; a.B = d.batch;
    a.zx = mid_zp; a.zy = y_zp; a.act_min = act_min; a.act_max = act_max;
    a.res = 0; a.raw = 0; a.ncls = 1; a.lsu = 0; a.w4 = nullptr; a.src = nullptr;
    a.full_count = kDwWarps;
    a.groups = 2; a.gwarps = 4;
    a.fold = p->rshift_max <= 53 ? (p->rshift_min >= 32 ? 1 : (p->narrow_ok ? 2 : 0)) : 0;
    DwFront& f = a.dw;
    f.taps = dwp->dw_taps; f.wsum = dwp->dw_wsum; f.bias = dwp->bias; f.mult = dwp->mult; f.rshift = dwp->rshift;
    f.tap_pitch = dd.c_pitch_in; f.c = dd.c; f.h = dd.h; f.w = dd.w;
    f.zx = x_zp; f.zy = mid_zp; f.act_min = mid_min; f.act_max = mid_max;
    f.gp = a.BK / 4;
    const int sd = dd.stride;
    // Tile: the box of output pixels (at most 128) that costs the depthwise warps least over the whole layer, among
    // those whose ring of input tiles fits beside at least two operand stages and one staging box per group.
    double best = 0.0;
    bool found = false;
    int bt[3] = {0, 0, 0};
    for (int tw = 2; tw <= std::min(a.W + (a.W & 1), kTileM); tw += 2) {
        if (tw > a.W + 1) break;
        for (int th = 1; th <= std::min(a.H, kTileM / tw); ++th) {
            const int tb = (tw >= a.W && th >= a.H) ? std::min(a.B, kTileM / (tw * th)) : 1;
            const int twin = (tw - 1) * sd + 3, thin = (th - 1) * sd + 3;
            if (twin > 256 || thin > 256) continue;
            const uint32_t sbytes = static_cast<uint32_t>(a.BK) * twin * thin * tb;
            const uint32_t sstride = (sbytes + 127u) & ~127u;
            if (make_layout(a.BK, a.BN, 2, 1, a.out_box, 2, 1, a.bres, 1, 0, 0, kDwinStages * sstride).total > static_cast<uint32_t>(kSmemBudget)) continue;
            const int pairs = tw / 2;
            const int spi = std::max(1, std::min(th, 32 * kDwWarps / std::max(1, f.gp * pairs * tb)));
            const int rps = (th + spi - 1) / spi;
            const int items = f.gp * pairs * tb * spi;
            const int iters = (items + 32 * kDwWarps - 1) / (32 * kDwWarps);
            const int64_t tiles = static_cast<int64_t>((a.W + tw - 1) / tw) * ((a.H + th - 1) / th) * ((a.B + tb - 1) / tb);
            const int64_t rounds = (tiles + h->num_sms - 1) / h->num_sms;
            // (per K block: the pieces' row steps, and the tile's input cells through the copy engine and shared memory)
            const double cost = static_cast<double>(rounds) * kblocks *
                                (iters * (rps + (sd == 1 ? 0.7 : 1.0)) + 0.8 + 0.02 * twin * thin * tb);
            if (!found || cost < best) {
                found = true;
                best = cost;
                bt[0] = tw; bt[1] = th; bt[2] = tb;
            }
        }
    }
    if (!found) return QTZ_ERR_UNSUPPORTED;
    a.tw = bt[0]; a.th = bt[1]; a.tb = bt[2];
    a.rows = a.tw * a.th * a.tb;
    a.tiles_w = (a.W + a.tw - 1) / a.tw;
    a.tiles_h = (a.H + a.th - 1) / a.th;
    const int64_t tiles = static_cast<int64_t>(a.tiles_w) * a.tiles_h * ((a.B + a.tb - 1) / a.tb);
    if (tiles > 0x7fffffff) return QTZ_ERR_UNSUPPORTED;
    a.num_tiles = static_cast<uint32_t>(tiles);
    a.m_tiles = static_cast<int32_t>(tiles);
    a.group_m = std::max(1, std::min(a.m_tiles, 16));
    a.dv_per_group = make_fastdiv(static_cast<uint32_t>(a.group_m));
    a.dv_group_m = make_fastdiv(static_cast<uint32_t>(a.group_m));
    a.dv_group_last = make_fastdiv(static_cast<uint32_t>(std::max(1, a.m_tiles % a.group_m)));
    a.dv_tiles_w = make_fastdiv(static_cast<uint32_t>(a.tiles_w));
    a.dv_tiles_h = make_fastdiv(static_cast<uint32_t>(a.tiles_h));
    f.twin = (a.tw - 1) * sd + 3;
    f.thin = (a.th - 1) * sd + 3;
    f.stage_bytes = static_cast<uint32_t>(a.BK) * f.twin * f.thin * a.tb;
    f.stage_stride = (f.stage_bytes + 127u) & ~127u;
    f.pairs = a.tw / 2;
    f.spi = std::max(1, std::min(a.th, 32 * kDwWarps / std::max(1, f.gp * f.pairs * a.tb)));
    f.rps = (a.th + f.spi - 1) / f.spi;
    f.items = f.gp * f.pairs * a.tb * f.spi;
    // ring depth and staging boxes from what is left of shared memory
    const uint32_t dwin_bytes = kDwinStages * f.stage_stride;
    a.obuf = 1;
    a.stages = 2;
    for (int ob = 2; ob >= 1 && a.obuf == 1; --ob)
        for (int st_ = 4; st_ >= 3; --st_)
            if (make_layout(a.BK, a.BN, st_, 1, a.out_box, 2, ob, a.bres, 1, 0, 0, dwin_bytes).total <= static_cast<uint32_t>(kSmemBudget)) {
                a.obuf = ob;
                a.stages = st_;
                break;
            }
    if (a.obuf == 1)
        for (int st_ = 4; st_ >= 2; --st_)
            if (make_layout(a.BK, a.BN, st_, 1, a.out_box, 2, 1, a.bres, 1, 0, 0, dwin_bytes).total <= static_cast<uint32_t>(kSmemBudget)) {
                a.stages = st_;
                break;
            }
    const uint32_t smem_bytes = make_layout(a.BK, a.BN, a.stages, 1, a.out_box, 2, a.obuf, a.bres, 1, 0, 0, dwin_bytes).total + 1024;
    if (smem_bytes > 227u * 1024u) return QTZ_ERR_UNSUPPORTED;

    CUtensorMap map_a, map_y;
    {
        const uint64_t pitch = static_cast<uint64_t>(dd.c_pitch_in);
        const uint64_t dims[4] = {static_cast<uint64_t>(dd.c), static_cast<uint64_t>(dd.w), static_cast<uint64_t>(dd.h),
                                  static_cast<uint64_t>(dd.batch)};
        const uint64_t strides[3] = {pitch, pitch * dd.w, pitch * dd.w * dd.h};
        const uint32_t box[4] = {static_cast<uint32_t>(a.BK), static_cast<uint32_t>(f.twin), static_cast<uint32_t>(f.thin),
                                 static_cast<uint32_t>(a.tb)};
        if (!encode_map(&map_a, x, 4, dims, strides, box, 0)) return QTZ_ERR_CUDA;
    }
    {
        const uint64_t opitch = static_cast<uint64_t>(d.c_pitch_out);
        const uint64_t dims[4] = {static_cast<uint64_t>(d.n), static_cast<uint64_t>(p->ow), static_cast<uint64_t>(p->oh),
                                  static_cast<uint64_t>(d.batch)};
        const uint64_t strides[3] = {opitch, opitch * p->ow, opitch * p->ow * p->oh};
        const uint32_t box[4] = {static_cast<uint32_t>(a.out_box), static_cast<uint32_t>(a.tw), static_cast<uint32_t>(a.th),
                                 static_cast<uint32_t>(a.tb)};
        if (!encode_map(&map_y, y, 4, dims, strides, box, a.out_box)) return QTZ_ERR_CUDA;
    }
    const int grid = static_cast<int>(std::min<int64_t>(a.num_tiles, h->num_sms));
    p->detail = std::string("tcgen05 pointwise weights:resident depthwise-front stride ") + std::to_string(sd) + " tile " +
                std::to_string(a.tw) + "x" + std::to_string(a.th) + "x" + std::to_string(a.tb);
    if (p->ev_start) QTZ_CUDA(h, cudaEventRecord(p->ev_start, st));
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(grid));
        cfg.blockDim = dim3(kThreadsTc);
        cfg.dynamicSmemBytes = smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        if (sd == 1) {
            QTZ_CUDA(h, cudaFuncSetAttribute(conv_tc_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            QTZ_CUDA(h, cudaLaunchKernelEx(&cfg, conv_tc_kernel<false, 1>, map_a, map_b, map_y, map_b, a));
        } else {
            QTZ_CUDA(h, cudaFuncSetAttribute(conv_tc_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            QTZ_CUDA(h, cudaLaunchKernelEx(&cfg, conv_tc_kernel<false, 2>, map_a, map_b, map_y, map_b, a));
        }
    }
    QTZ_LAUNCH_CHECK(h, "conv_tc_kernel (depthwise front)");
    if (p->ev_stop) QTZ_CUDA(h, cudaEventRecord(p->ev_stop, st));
    return QTZ_OK;
}
