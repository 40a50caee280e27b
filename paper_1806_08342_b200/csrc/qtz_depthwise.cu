// 3x3 depthwise convolution (stride 1 or 2, pad 1, depth multiplier 1) on the CUDA cores.
//
// Depthwise is not a dense contraction (each channel has its own 9 weights), so it is bound
// by HBM traffic -- 1 byte in and 1 byte out per output at stride 1 -- provided the
// instruction count per output stays low and nothing serialises the block.  Design:
//  * persistent blocks walk over tiles (images x rows x columns x channel chunk).  Warp 0 is a
//    producer: one lane fetches whole input tiles with TMA box copies (halo included,
//    out-of-image pixels zero-filled) into a ring of shared-memory stages and publishes the
//    tile's coordinates beside it; the other warps consume.  Stages are handed over through
//    mbarriers (full: TMA bytes landed; empty: one arrival per consumer warp), so there is no
//    block-wide barrier anywhere in the steady state;
//  * real zero is the code z_x, not 0, so tiles that touch the image border overwrite their
//    out-of-image cells with z_x before use (a barrier among the consumer warps only); then
//    acc = bias - z_x sum(w) + sum x w holds for every output (Eq. 5-6 with K = 9, every tap
//    "valid");
//  * a thread owns 4 channels x 2 adjacent output columns and walks down the tile; each input
//    row is read once from shared memory (four or five 4-byte loads), byte-transposed in
//    registers (PRMT) so that one register holds pixels (w0-1 .. w0+2) of ONE channel, and kept
//    for the three output rows it feeds; a filter row is then one dp4a against the packed
//    weights (k0,k1,k2,0) for column w0 and (0,k0,k1,k2) for column w0+1, both forms resident
//    in registers;
//  * uint8 weights arrive shifted to int8 with their zero point; the extra -z_w sum(x) term
//    costs one more dp4a per window against (1,1,1,0);
//  * requantisation for right shifts of 32 and more is one 64-bit multiply-add (the addend holds
//    the rounding constant, the output offset and the bias / zero-point constant times the
//    multiplier, so the accumulators start from zero), one shift of the high word, and
//    cvt.pack.sat to bytes; the clamp is a fused min/max-with-zero, left out altogether when
//    the activation range is the whole byte (the saturating pack already clamps).
// Every wait on an mbarrier is bounded; on expiry the kernel records a status word and returns.
#include <algorithm>
#include <new>
#include <string>

#include "qtz_dw_math.cuh"
#include "qtz_plan.cuh"
#include "qtz_ptx.cuh"

using namespace qtz_ptx;
using namespace qtz_dw;

namespace {

constexpr int kDwMaxThreads = 256;                      // one producer warp + up to seven consumer warps
constexpr int kDwMaxConsumers = kDwMaxThreads - 32;
constexpr int kDwMaxStages = 4;
constexpr int kDwSmemPerSm = 227 * 1024;
constexpr int kDwRegsPerThread = 128;                   // what __launch_bounds__(256, 2) allows
constexpr int kDwWarpsToSaturate = 21;                  // consumer warps per SM beyond which more residency buys nothing

struct DwArgs {
    uint8_t* y;
    int32_t* y_raw;         // kModeRaw: int32 accumulators [pixel][c] instead of uint8 codes
    const uint32_t* taps;   // [3][tap_pitch]: per filter row and channel, bytes (k0, k1, k2, 0) as int8
    const int32_t* wsum;    // [tap_pitch]: sum of the nine int8 codes
    const int32_t* bias;    // padded beyond c
    const int32_t* mult;
    const int32_t* rshift;
    int32_t* status;
    long long wait_budget;
    int batch, h, w_, c, tap_pitch, yp, oh, ow;
    int cb, tw, th, nb, twin, thin;      // tile: channels, output columns / rows, images, input columns / rows
    int gp, pairs, slots, spi, rps;      // thread mapping: channel groups, column pairs, row slots, slots per image, rows per slot
    int units;                           // nb * spi pieces of work per tile, taken by the slots in turn
    int consumers, stages;
    int tiles_w, tiles_h, c_chunks, b_tiles;
    int64_t num_tiles;
    uint32_t tile_bytes, buf_stride;
    int zx, zw, zy, act_min, act_max;
};

// Where a thread writes: its first column's pixel, the byte offset to the second column
// (0 when that column is outside the image: the store is skipped) and the pitch of an output row.
struct OutCursor {
    uint8_t* p;
    int32_t* raw;
    int col2;        // byte offset of the second column (0 when it is outside the image)
    int row;         // byte offset of the next output row
    int raw_c, raw_row;
    bool second;
    int valid_ch;    // channels of this thread that exist (raw output only)
};

template <int kStride, bool kAsym, int kMode, bool kClamp>
__device__ __forceinline__ void emit_row(const RowState<kStride>& r0, const RowState<kStride>& r1, const RowState<kStride>& r2,
                                         const ChanConst<kMode>& k, OutCursor& o)
{
    int32_t acc[2][4];
    mac3<kStride, kAsym, kMode>(r0, r1, r2, k, acc);
    if (kMode == kModeRaw) {   // calibration: the accumulators themselves
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            if (ch < o.valid_ch) {
                o.raw[ch] = acc[0][ch];
                if (o.second) o.raw[o.raw_c + ch] = acc[1][ch];
            }
        }
        o.raw += o.raw_row;
    } else {
        const uint32_t y0 = requant_pixel<kMode, kClamp>(acc[0], k);
        const uint32_t y1 = requant_pixel<kMode, kClamp>(acc[1], k);
        *reinterpret_cast<uint32_t*>(o.p + o.col2) = y1;   // col2 = 0 when the second column is outside: overwritten next
        *reinterpret_cast<uint32_t*>(o.p) = y0;
        o.p += o.row;
    }
}

struct TileCoord {
    int cc, b, h0, w0;   // channel chunk, first image, first output row / column
};

// The channel chunk is the fastest index: blocks that run side by side read neighbouring
// chunks of the same pixels.  The grid is a multiple of the chunk count, so a block keeps its
// chunk (and the per-channel constants in its registers) for its whole life.
__device__ __forceinline__ TileCoord decode_tile(const DwArgs& a, int tile)
{
    TileCoord t;
    t.cc = tile % a.c_chunks; tile /= a.c_chunks;
    t.w0 = (tile % a.tiles_w) * a.tw; tile /= a.tiles_w;
    t.h0 = (tile % a.tiles_h) * a.th; tile /= a.tiles_h;
    t.b = tile * a.nb;
    return t;
}

template <int kStride, bool kAsym, int kMode, bool kClamp>
__global__ void __launch_bounds__(kDwMaxThreads, 2)
depthwise3x3_kernel(const __grid_constant__ CUtensorMap map_x, const DwArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base_addr = (smem_u32(smem_raw) + 127u) & ~127u;
    uint8_t* const smem = smem_raw + (base_addr - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bars[2 * kDwMaxStages];   // full[stage], then empty[stage]
    __shared__ int4 coords[kDwMaxStages];                       // (cc, b, h0, w0) of the tile in each stage
    const uint32_t full0 = smem_u32(&bars[0]);
    const uint32_t empty0 = smem_u32(&bars[kDwMaxStages]);
    const int stages = a.stages;
    const int num_tiles = static_cast<int>(a.num_tiles);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, a.consumers / 32);
        }
        fence_barrier_init();
        prefetch_tensormap(&map_x);
        grid_launch_dependents();     // the next kernel may be scheduled as this one's blocks leave
    }
    __syncthreads();
    // started, perhaps, before the previous kernel of the stream has finished (programmatic dependent launch): its
    // output is this kernel's input, and this kernel's output may alias what it still reads
    grid_dependency_wait();

    if (threadIdx.x < 32) {
        // ---- producer: lane 0 streams tiles into the ring ----
        if (threadIdx.x != 0) return;
        int stage = 0;
        uint32_t round = 0;
        for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
            if (round > 0 && !mbar_wait(empty0 + 8 * stage, (round - 1) & 1, a.wait_budget, 256u)) {
                if (atomicCAS(a.status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) a.status[1] = QTZ_SITE_SMEM_EMPTY;
                return;
            }
            const TileCoord t = decode_tile(a, tile);
            coords[stage] = make_int4(t.cc, t.b, t.h0, t.w0);   // published by the arrive below
            mbar_arrive_expect_tx(full0 + 8 * stage, a.tile_bytes);
            tma_load_4d(base_addr + stage * a.buf_stride, &map_x, full0 + 8 * stage, t.cc * a.cb, t.w0 * kStride - 1,
                        t.h0 * kStride - 1, t.b);
            if (++stage == stages) { stage = 0; ++round; }
        }
        return;
    }

    // ---- consumers ----
    const int tid = threadIdx.x - 32;
    const int g = tid % a.gp;
    const int pr = (tid / a.gp) % a.pairs;
    const int sl = tid / (a.gp * a.pairs);
    const bool in_slot = sl < a.slots;

    ChanConst<kMode> k;
    k.off = a.zy - a.act_min;
    k.span = a.act_max - a.act_min;
    k.lo4 = 0x01010101u * static_cast<uint32_t>(a.act_min);
    k.zw = a.zw;
    const uint32_t fill = 0x01010101u * static_cast<uint32_t>(a.zx);
    int loaded_cc = -1;
    const int row_bytes = a.twin * a.cb;
    WinOffsets wo;
    wo.o1 = a.cb; wo.o2 = 2 * a.cb; wo.o3 = 3 * a.cb; wo.o4 = 4 * a.cb;
    const uint32_t thread_cell = (2 * pr * kStride) * a.cb + 4 * g;   // the thread's window inside a tile row

    int stage = 0;
    uint32_t round = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        if (!mbar_wait(full0 + 8 * stage, round & 1, a.wait_budget)) {
            if (atomicCAS(a.status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) a.status[1] = QTZ_SITE_TMA_FULL;
            return;
        }
        const int4 tc = coords[stage];
        TileCoord t;
        t.cc = tc.x; t.b = tc.y; t.h0 = tc.z; t.w0 = tc.w;

        const int c0 = t.cc * a.cb + 4 * g;
        const bool worker = in_slot && c0 < a.c;   // groups entirely beyond the last channel idle
        if (worker && t.cc != loaded_cc) {         // per-channel constants of this channel chunk
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint4 w = __ldg(reinterpret_cast<const uint4*>(a.taps + static_cast<int64_t>(i) * a.tap_pitch + c0));
                k.wa[i][0] = w.x; k.wa[i][1] = w.y; k.wa[i][2] = w.z; k.wa[i][3] = w.w;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) k.wb[i][ch] = k.wa[i][ch] << 8;
            }
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                const int32_t r = kMode == kModeRaw ? 40 : __ldg(a.rshift + c0 + ch);   // raw output has no multipliers
                const int32_t base = __ldg(a.bias + c0 + ch) - a.zx * __ldg(a.wsum + c0 + ch) + 9 * a.zx * a.zw;
                k.m[ch] = kMode == kModeRaw ? 0 : __ldg(a.mult + c0 + ch);
                k.sh[ch] = kMode == kModeFast ? r - 32 : r;
                if (kMode == kModeFast)   // exact in 64-bit wrap-around arithmetic: the true sum fits
                    k.add[kMode == kModeFast ? ch : 0] = (static_cast<int64_t>(2 * k.off + 1) << (r - 1)) + static_cast<int64_t>(base) * k.m[ch];
                else
                    k.base[kMode == kModeFast ? 0 : ch] = base;
            }
            loaded_cc = t.cc;
        }

        uint8_t* const tile_s = smem + stage * a.buf_stride;
        // padding is real zero = code z_x: overwrite the cells TMA zero-filled outside the image
        const int ih0 = t.h0 * kStride - 1, iw0 = t.w0 * kStride - 1;
        const bool border = a.zx != 0 && (ih0 < 0 || iw0 < 0 || ih0 + a.thin > a.h || iw0 + a.twin > a.w_);
        if (border) {
            const int rows_in = min(a.thin, a.h - ih0);        // tile rows [first_row, rows_in) are inside the image
            const int first_row = ih0 < 0 ? 1 : 0;
            const int cols_in = min(a.twin, a.w_ - iw0);        // tile columns [first_col, cols_in) are inside
            const int first_col = iw0 < 0 ? 1 : 0;
            const int lane8 = 8 * (tid & 31), warp_id = tid >> 5, warps = a.consumers >> 5;
            for (int img = 0; img < a.nb; ++img) {
                uint8_t* const img_s = tile_s + img * a.thin * row_bytes;
                if (first_row)                                  // the row above the image
                    for (int i = 8 * tid; i < row_bytes; i += 8 * a.consumers) *reinterpret_cast<uint2*>(img_s + i) = make_uint2(fill, fill);
                for (int ri = rows_in; ri < a.thin; ++ri)       // rows below the image
                    for (int i = 8 * tid; i < row_bytes; i += 8 * a.consumers)
                        *reinterpret_cast<uint2*>(img_s + ri * row_bytes + i) = make_uint2(fill, fill);
                if (first_col + a.twin - cols_in > 0) {         // the left column and / or the right columns
                    for (int ri = first_row + warp_id; ri < rows_in; ri += warps) {
                        uint8_t* row = img_s + ri * row_bytes;
                        if (first_col)
                            for (int i = lane8; i < a.cb; i += 256) *reinterpret_cast<uint2*>(row + i) = make_uint2(fill, fill);
                        for (int i = lane8; i < (a.twin - cols_in) * a.cb; i += 256)
                            *reinterpret_cast<uint2*>(row + cols_in * a.cb + i) = make_uint2(fill, fill);
                    }
                }
            }
            named_barrier(1, a.consumers);
        }

        const int ow0 = t.w0 + 2 * pr;
        if (worker && ow0 < a.ow) {
            OutCursor o;
            o.second = ow0 + 1 < a.ow;
            o.col2 = o.second ? a.yp : 0;
            o.row = a.ow * a.yp;
            o.raw_c = a.c;
            o.raw_row = a.ow * a.c;
            o.valid_ch = a.c - c0;
            const uint32_t tile_cell = base_addr + stage * a.buf_stride + thread_cell;
            for (int unit = sl; unit < a.units; unit += a.slots) {
                int img = 0, part = unit;
                if (a.nb > 1) { img = unit / a.spi; part = unit - img * a.spi; }
                if (t.b + img >= a.batch) break;
                const int r_begin = part * a.rps;
                int n = min(min(a.th, r_begin + a.rps), a.oh - t.h0) - r_begin;   // output rows of this unit
                if (n <= 0) continue;
                uint32_t cell = tile_cell + (img * a.thin + r_begin * kStride) * row_bytes;
                const int64_t first_px = (static_cast<int64_t>(t.b + img) * a.oh + t.h0 + r_begin) * a.ow + ow0;
                o.p = a.y + first_px * a.yp + c0;
                o.raw = a.y_raw + first_px * a.c + c0;

                if (kStride == 1) {
                    // three input rows stay in registers and rotate: tile rows r, r+1, r+2 feed output row r
                    RowState<1> r0, r1, r2;
                    load_row<1>(cell, wo, r0); cell += row_bytes;
                    load_row<1>(cell, wo, r1); cell += row_bytes;
                    for (; n >= 3; n -= 3) {
                        load_row<1>(cell, wo, r2); cell += row_bytes;
                        emit_row<1, kAsym, kMode, kClamp>(r0, r1, r2, k, o);
                        load_row<1>(cell, wo, r0); cell += row_bytes;
                        emit_row<1, kAsym, kMode, kClamp>(r1, r2, r0, k, o);
                        load_row<1>(cell, wo, r1); cell += row_bytes;
                        emit_row<1, kAsym, kMode, kClamp>(r2, r0, r1, k, o);
                    }
                    if (n >= 1) {
                        load_row<1>(cell, wo, r2); cell += row_bytes;
                        emit_row<1, kAsym, kMode, kClamp>(r0, r1, r2, k, o);
                        if (n == 2) {
                            load_row<1>(cell, wo, r0);
                            emit_row<1, kAsym, kMode, kClamp>(r1, r2, r0, k, o);
                        }
                    }
                } else {
                    // stride 2: tile rows 2r, 2r+1, 2r+2; the last one is the next output row's first
                    RowState<2> top, mid, bot;
                    load_row<2>(cell, wo, top); cell += row_bytes;
                    for (; n >= 2; n -= 2) {
                        load_row<2>(cell, wo, mid); cell += row_bytes;
                        load_row<2>(cell, wo, bot); cell += row_bytes;
                        emit_row<2, kAsym, kMode, kClamp>(top, mid, bot, k, o);
                        load_row<2>(cell, wo, mid); cell += row_bytes;
                        load_row<2>(cell, wo, top); cell += row_bytes;
                        emit_row<2, kAsym, kMode, kClamp>(bot, mid, top, k, o);
                    }
                    if (n == 1) {
                        load_row<2>(cell, wo, mid); cell += row_bytes;
                        load_row<2>(cell, wo, bot);
                        emit_row<2, kAsym, kMode, kClamp>(top, mid, bot, k, o);
                    }
                }
            }
        }
        // hand the stage back: this warp's reads (and border writes) are done
        if (border) fence_proxy_async_smem();   // generic-proxy writes must not be overtaken by the refill
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(empty0 + 8 * stage);
        if (++stage == stages) { stage = 0; ++round; }
    }
}

using DwKernel = void (*)(const CUtensorMap, const DwArgs);

template <int kStride, bool kAsym>
DwKernel pick_mode(int mode, bool clamp)
{
    switch (mode) {
    case kModeFast: return clamp ? depthwise3x3_kernel<kStride, kAsym, kModeFast, true> : depthwise3x3_kernel<kStride, kAsym, kModeFast, false>;
    case kModeRaw: return depthwise3x3_kernel<kStride, kAsym, kModeRaw, false>;
    default: return depthwise3x3_kernel<kStride, kAsym, kModeGeneral, true>;
    }
}

DwKernel pick_kernel(int stride, bool asym, int mode, bool clamp)
{
    if (stride == 1) return asym ? pick_mode<1, true>(mode, clamp) : pick_mode<1, false>(mode, clamp);
    return asym ? pick_mode<2, true>(mode, clamp) : pick_mode<2, false>(mode, clamp);
}

}  // namespace

struct qtz_dw_state {
    DwArgs args{};
    uint32_t smem_bytes = 0;
    int grid = 0;
    int threads = 0;
};

// Chooses the tile (channel chunk, output columns, rows and images), the thread mapping and the
// grid.  Candidates (rows per tile, images per tile) are ranked by a model of the time of the
// busiest SM: rounds of tiles per block x blocks per SM x consumer warps x instructions a thread
// spends on one tile (about 64 per output row of its two columns, 24 per slot start for the two
// halo rows, a fixed hand-over cost per tile).
qtz_status qtz_depthwise_prepare(qtz_plan* p)
{
    const qtz_conv_desc& d = p->d;
    qtz_dw_state* s = new (std::nothrow) qtz_dw_state();
    if (!s) return QTZ_ERR_INVALID_ARG;
    p->dw = s;
    DwArgs& a = s->args;
    const int st = d.stride;
    a.batch = d.batch; a.h = d.h; a.w_ = d.w; a.c = d.c; a.tap_pitch = d.c_pitch_in; a.yp = d.c_pitch_out;
    a.oh = p->oh; a.ow = p->ow;
    // channel chunk: at most 128 channels, a multiple of 16 (TMA rows are 16-byte multiples)
    a.c_chunks = (d.c + 127) / 128;
    a.cb = ((d.c + a.c_chunks - 1) / a.c_chunks + 15) / 16 * 16;
    a.gp = a.cb / 4;
    // columns: as many pairs as fit the consumer threads and the image, split evenly over the tiles of a row
    const int all_pairs = (p->ow + 1) / 2;
    const int max_pairs = std::max(1, std::min(kDwMaxConsumers / a.gp, all_pairs));
    a.tiles_w = (all_pairs + max_pairs - 1) / max_pairs;
    a.pairs = (all_pairs + a.tiles_w - 1) / a.tiles_w;
    a.tw = 2 * a.pairs;
    a.twin = (a.tw - 1) * st + 3;
    a.tiles_w = (p->ow + a.tw - 1) / a.tw;
    if (a.twin > 256) return QTZ_ERR_UNSUPPORTED;
    const int slots_max = std::max(1, kDwMaxConsumers / (a.gp * a.pairs));
    const int sms = p->h->num_sms;

    double best = 0.0;
    bool found = false;
    qtz_dw_state pick;
    for (int stages = 2; stages <= 3; ++stages) {
        for (int th = 1; th <= p->oh; ++th) {
            const int tiles_h = (p->oh + th - 1) / th;
            if ((p->oh + tiles_h - 1) / tiles_h != th) continue;   // the same split with fewer rows per tile exists
            const int thin = (th - 1) * st + 3;
            if (thin > 256) break;
            const int64_t bytes1 = static_cast<int64_t>(thin) * a.twin * a.cb;
            const int nb_max = (tiles_h == 1 && a.tiles_w == 1) ? std::min(d.batch, 64) : 1;
            for (int nb = 1; nb <= nb_max; ++nb) {
                const int64_t tile_bytes = bytes1 * nb;
                const int64_t buf_stride = (tile_bytes + 127) & ~static_cast<int64_t>(127);
                const int64_t smem = stages * buf_stride + 128;
                if (smem + 1024 > kDwSmemPerSm / 2) break;          // at least two blocks per SM
                int spi, slots;
                if (nb == 1) { spi = std::min(slots_max, th); slots = spi; }
                else if (slots_max >= nb) { spi = std::min(th, slots_max / nb); slots = spi * nb; }
                else { spi = 1; slots = slots_max; }
                const int rps = (th + spi - 1) / spi;
                const int units = nb * spi;
                const int iters = (units + slots - 1) / slots;
                const int consumers = (a.gp * a.pairs * slots + 31) / 32 * 32;
                const int threads = consumers + 32;
                int bps = static_cast<int>(kDwSmemPerSm / (smem + 1024));
                bps = std::min(bps, 65536 / (threads * kDwRegsPerThread));
                bps = std::min(bps, 2048 / threads);
                bps = std::min(bps, 8);
                if (bps < 1) continue;
                const int b_tiles = (d.batch + nb - 1) / nb;
                const int64_t tiles = static_cast<int64_t>(a.c_chunks) * b_tiles * tiles_h * a.tiles_w;
                int64_t grid = std::min<int64_t>(tiles, static_cast<int64_t>(sms) * bps);
                if (grid > a.c_chunks) grid -= grid % a.c_chunks;   // a block keeps its channel chunk
                const int64_t rounds = (tiles + grid - 1) / grid;
                const int64_t blocks_on_sm = (grid + sms - 1) / sms;
                const double per_tile = iters * ((st == 2 ? 84.0 : 64.0) * rps + 24.0 * st) + 80.0;
                // work of the busiest SM, divided by the rate its resident warps reach
                const double resident = static_cast<double>(blocks_on_sm) * (consumers / 32);
                const double rate = std::min(resident, static_cast<double>(kDwWarpsToSaturate));
                const double cost = static_cast<double>(rounds) * resident * per_tile / rate *
                                    (stages == 2 ? 1.0 : 0.98);   // a deeper ring hides more load latency
                if (!found || cost < best) {
                    found = true;
                    best = cost;
                    pick.args = a;
                    DwArgs& b = pick.args;
                    b.th = th; b.thin = thin; b.tiles_h = tiles_h; b.nb = nb; b.spi = spi; b.slots = slots; b.rps = rps;
                    b.units = units; b.consumers = consumers; b.stages = stages; b.b_tiles = b_tiles; b.num_tiles = tiles;
                    b.tile_bytes = static_cast<uint32_t>(tile_bytes);
                    b.buf_stride = static_cast<uint32_t>(buf_stride);
                    pick.smem_bytes = static_cast<uint32_t>(smem);
                    pick.grid = static_cast<int>(grid);
                    pick.threads = threads;
                }
            }
        }
    }
    if (!found) return QTZ_ERR_UNSUPPORTED;
    *s = pick;
    a.taps = p->dw_taps; a.wsum = p->dw_wsum; a.bias = p->bias; a.mult = p->mult; a.rshift = p->rshift;
    a.status = p->h->status_dev;
    a.wait_budget = p->h->wait_budget;
    a.zw = p->w_zp_signed;
    // the attribute is per device: set it for this plan's device every time (cheap, and safe from any host thread)
    for (int stride = 1; stride <= 2; ++stride)
        for (int asym = 0; asym < 2; ++asym)
            for (int mode = 0; mode < kNumModes; ++mode)
                for (int clamp = 0; clamp < 2; ++clamp) {
                    const cudaError_t e = cudaFuncSetAttribute(pick_kernel(stride, asym != 0, mode, clamp != 0),
                                                               cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                               kDwSmemPerSm / 2);
                    if (e != cudaSuccess) return qtz_cuda_fail(p->h, e, "cudaFuncSetAttribute(depthwise3x3_kernel)");
                }
    return QTZ_OK;
}

void qtz_depthwise_release(qtz_plan* p)
{
    delete p->dw;
    p->dw = nullptr;
}

qtz_status qtz_depthwise_launch(qtz_plan* p, const uint8_t* x, int32_t x_zp, uint8_t* y, int32_t y_zp, int32_t act_min,
                                int32_t act_max, cudaStream_t st)
{
    const qtz_conv_desc& d = p->d;
    DwArgs a = p->dw->args;
    const bool raw = d.outkind == QTZ_OUT_S32_RAW;
    a.y = raw ? nullptr : y;
    a.y_raw = raw ? reinterpret_cast<int32_t*>(y) : nullptr;
    a.zx = x_zp; a.zy = y_zp; a.act_min = act_min; a.act_max = act_max;
    a.wait_budget = p->h->wait_budget;
    CUtensorMap map;
    const uint64_t pitch = static_cast<uint64_t>(d.c_pitch_in);
    const uint64_t dims[4] = {static_cast<uint64_t>(d.c), static_cast<uint64_t>(d.w), static_cast<uint64_t>(d.h),
                              static_cast<uint64_t>(d.batch)};
    const uint64_t strides[3] = {pitch, pitch * d.w, pitch * d.w * d.h};
    const uint32_t box[4] = {static_cast<uint32_t>(a.cb), static_cast<uint32_t>(a.twin), static_cast<uint32_t>(a.thin),
                             static_cast<uint32_t>(a.nb)};
    if (!qtz_encode_u8_map(&map, x, 4, dims, strides, box, 0)) {
        p->h->last_error = "cuTensorMapEncodeTiled failed for the depthwise input";
        return QTZ_ERR_CUDA;
    }
    // requantisation form by the layer's right shifts: the fast form for 32..53, else the general one
    const int mode = raw ? kModeRaw : ((p->rshift_max > 53 || p->rshift_min < 32) ? kModeGeneral : kModeFast);
    const bool clamp = !(act_min == 0 && act_max == 255);
    const DwKernel kernel = pick_kernel(d.stride, p->w_zp_signed != 0, mode, clamp);
    p->detail = std::string("depthwise tile ") + std::to_string(a.tw) + "x" + std::to_string(a.th) + "x" + std::to_string(a.nb) +
                " stages:" + std::to_string(a.stages);
    if (p->ev_start) QTZ_CUDA(p->h, cudaEventRecord(p->ev_start, st));
    {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(p->dw->grid));
        cfg.blockDim = dim3(static_cast<unsigned>(p->dw->threads));
        cfg.dynamicSmemBytes = p->dw->smem_bytes;
        cfg.stream = st;
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at.val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = &at;
        cfg.numAttrs = 1;
        QTZ_CUDA(p->h, cudaLaunchKernelEx(&cfg, kernel, map, a));
    }
    QTZ_LAUNCH_CHECK(p->h, "depthwise3x3_kernel");
    if (p->ev_stop) QTZ_CUDA(p->h, cudaEventRecord(p->ev_stop, st));
    return QTZ_OK;
}
