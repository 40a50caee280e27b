// 3x3 depthwise convolution (stride 1 or 2, pad 1, depth multiplier 1) on the CUDA cores.
//
// Depthwise is not a dense contraction (each channel has its own 9 weights), so it is bound
// by HBM traffic -- 1 byte in and 1 byte out per output at stride 1 -- provided the
// instruction count per output stays low and enough bytes are in flight.  Design:
//  * persistent blocks walk over tiles (rows x columns x channel chunk of one image); thread 0
//    fetches the input tile of the NEXT tile with one TMA box copy (halo included, out-of-image
//    pixels zero-filled) into the other of two shared-memory buffers while the block computes
//    the current one: no per-thread global loads, no address arithmetic per pixel;
//  * real zero is the code z_x, not 0, so tiles that touch the image border overwrite their
//    out-of-image cells with z_x before use; then acc = bias - z_x sum(w) + sum x w holds for
//    every output (Eq. 5-6 with K = 9, every tap "valid");
//  * a thread owns 8 channels x 2 adjacent output columns and walks down the tile; each input
//    row is read once from shared memory (four 8-byte loads), byte-transposed in registers
//    (PRMT) so that one register holds pixels (w0-1 .. w0+2) of ONE channel, and kept for the
//    three output rows it feeds; a filter row is then one dp4a against the packed weights
//    (k0,k1,k2,0) for column w0 and (0,k0,k1,k2) for column w0+1;
//  * uint8 weights arrive shifted to int8 with their zero point; the extra -z_w sum(x) term
//    costs one more dp4a per window against (1,1,1,0);
//  * requantisation is one 64-bit multiply-add per value (the rounding constant and the output
//    offset, folded, live in the high word for shifts >= 33), a shift of the high word, one
//    fused min/max-with-zero for the clamp, and cvt.pack.sat to bytes.
// Every wait on an mbarrier is bounded; on expiry the kernel records a status word and returns.
#include <algorithm>
#include <new>

#include "qtz_plan.cuh"
#include "qtz_ptx.cuh"

using namespace qtz_ptx;

namespace {

constexpr int kDwThreads = 256;
constexpr int kDwSmemLimit = 200 * 1024;

struct DwArgs {
    uint8_t* y;
    int32_t* y_raw;         // when set: int32 accumulators [pixel][c] instead of uint8 codes
    const uint32_t* taps;   // [3][tap_pitch]: per filter row and channel, bytes (k0, k1, k2, 0) as int8
    const int32_t* wsum;    // [tap_pitch]: sum of the nine int8 codes
    const int32_t* bias;    // padded beyond c
    const int32_t* mult;
    const int32_t* rshift;
    int32_t* status;
    long long wait_budget;
    int batch, h, w_, c, tap_pitch, yp, oh, ow;
    int cb, tw, th, twin, thin;          // tile: channels, output columns / rows, input columns / rows
    int gp, pairs, slots, rps;           // thread mapping: channel groups, column pairs, row slots, rows per slot
    int tiles_w, tiles_h, c_chunks;
    int64_t num_tiles;
    uint32_t tile_bytes, buf_stride;
    int zx, zw, zy, act_min, act_max;
};

__device__ __forceinline__ int32_t dp4a_us(uint32_t a, uint32_t b, int32_t c)
{
    int32_t d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// d = (c << 16) | (sat_u8(a) << 8) | sat_u8(b)
__device__ __forceinline__ uint32_t pack_sat_u8(int32_t a, int32_t b, uint32_t c)
{
    uint32_t d;
    asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// 4x4 byte transpose: a_j holds 4 channels of pixel j; t[ch] receives 4 pixels of channel ch.
__device__ __forceinline__ void transpose4(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t* t)
{
    const uint32_t lo01 = __byte_perm(a0, a1, 0x5140), hi01 = __byte_perm(a0, a1, 0x7362);
    const uint32_t lo23 = __byte_perm(a2, a3, 0x5140), hi23 = __byte_perm(a2, a3, 0x7362);
    t[0] = __byte_perm(lo01, lo23, 0x5410);
    t[1] = __byte_perm(lo01, lo23, 0x7632);
    t[2] = __byte_perm(hi01, hi23, 0x5410);
    t[3] = __byte_perm(hi01, hi23, 0x7632);
}

// One input row as the two output columns of a thread see it, 8 channels.
//   stride 1: t[ch] = pixels (w0-1, w0, w0+1, w0+2): column w0 reads bytes 0..2, column w0+1 bytes 1..3
//   stride 2: t[ch] = inputs (2w0, .., 2w0+3): column w0+1 reads bytes 1..3;
//             l[ch] = inputs (2w0-1, 2w0, 2w0+1, -): column w0 reads bytes 0..2
template <int kStride>
struct RowState {
    uint32_t t[8];
    uint32_t l[kStride == 2 ? 8 : 1];
};

// Reads the thread's window of one tile row from shared memory.  `cell` addresses the first
// window pixel of that row (8 channels of the thread), `cb` is the pixel pitch in bytes.
template <int kStride>
__device__ __forceinline__ void load_row(const uint8_t* cell, int cb, RowState<kStride>& r)
{
    constexpr int kCols = kStride == 1 ? 4 : 5;
    uint2 raw[kCols];
#pragma unroll
    for (int j = 0; j < kCols; ++j) raw[j] = *reinterpret_cast<const uint2*>(cell + j * cb);
    if (kStride == 1) {
        transpose4(raw[0].x, raw[1].x, raw[2].x, raw[3].x, r.t);
        transpose4(raw[0].y, raw[1].y, raw[2].y, raw[3].y, r.t + 4);
    } else {
        transpose4(raw[1].x, raw[2].x, raw[3].x, raw[4].x, r.t);
        transpose4(raw[1].y, raw[2].y, raw[3].y, raw[4].y, r.t + 4);
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
            r.l[ch] = __byte_perm(raw[0].x, r.t[ch], 0x6540 | ch);
            r.l[4 + ch] = __byte_perm(raw[0].y, r.t[4 + ch], 0x6540 | ch);
        }
    }
}

// Adds one filter row (w1[ch] = bytes (k0,k1,k2,0)) applied to one input row.  With kInit the
// accumulators start from `base` (bias and zero-point constant) instead of their old value.
template <int kStride, bool kAsym, bool kInit>
__device__ __forceinline__ void mac_row(const RowState<kStride>& r, const uint32_t (&w1)[8], const int32_t (&base)[8],
                                        int32_t (&acc)[2][8], int32_t (&xs)[2][8])
{
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
        const uint32_t w2 = w1[ch] << 8;   // (0,k0,k1,k2)
        const uint32_t first = kStride == 1 ? r.t[ch] : r.l[kStride == 2 ? ch : 0];
        acc[0][ch] = dp4a_us(first, w1[ch], kInit ? base[ch] : acc[0][ch]);
        acc[1][ch] = dp4a_us(r.t[ch], w2, kInit ? base[ch] : acc[1][ch]);
        if (kAsym) {
            xs[0][ch] = dp4a_us(first, 0x00010101u, kInit ? 0 : xs[0][ch]);
            xs[1][ch] = dp4a_us(r.t[ch], 0x01010100u, kInit ? 0 : xs[1][ch]);
        }
    }
}

struct Requant {
    int32_t m[8];
    int32_t sh[8];      // fast form: r - 32;  general form: r
    int32_t addhi[8];   // fast form, r >= 33: high word of 2^(r-1) + ((z_y - act_min) << r) (its low word is zero)
    int64_t add[8];     // fast form, r >= 32: the same constant in full
    uint32_t lo4;       // act_min in every byte
    int32_t span;       // act_max - act_min
    int32_t zy, lo;
};

// Requantises 8 channels of one pixel and returns them as two packed words.  The clamp is done
// relative to act_min: max(min(y - act_min, span), 0) is a single instruction, act_min is added
// back to all four bytes of a packed word at once.
template <int kFast>
__device__ __forceinline__ uint2 requant_pixel(const int32_t (&v)[8], const Requant& q)
{
    int32_t y[8];
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
        if (kFast != 0) {   // 32 (33) <= r <= 53: floor((v m + addend) / 2^r) = hi32(v m + addend) >> (r - 32)
            const int64_t p = static_cast<int64_t>(v[ch]) * q.m[ch] +
                              (kFast == 1 ? static_cast<int64_t>(q.addhi[ch]) << 32 : q.add[ch]);
            y[ch] = __vimin_s32_relu(static_cast<int32_t>(p >> 32) >> q.sh[ch], q.span);
        } else {
            const int64_t p = static_cast<int64_t>(v[ch]) * q.m[ch] + (static_cast<int64_t>(1) << (q.sh[ch] - 1));
            const int64_t s = (p >> q.sh[ch]) + (q.zy - q.lo);
            y[ch] = static_cast<int32_t>(min(max(s, static_cast<int64_t>(0)), static_cast<int64_t>(q.span)));
        }
    }
    uint2 o;
    o.x = pack_sat_u8(y[1], y[0], pack_sat_u8(y[3], y[2], 0u)) + q.lo4;
    o.y = pack_sat_u8(y[5], y[4], pack_sat_u8(y[7], y[6], 0u)) + q.lo4;
    return o;
}

struct TileCoord {
    int cc, b, h0, w0;   // channel chunk, image, first output row / column
};

__device__ __forceinline__ TileCoord decode_tile(const DwArgs& a, int64_t tile)
{
    TileCoord t;
    t.w0 = static_cast<int>(tile % a.tiles_w) * a.tw; tile /= a.tiles_w;
    t.h0 = static_cast<int>(tile % a.tiles_h) * a.th; tile /= a.tiles_h;
    t.b = static_cast<int>(tile % a.batch);
    t.cc = static_cast<int>(tile / a.batch);
    return t;
}

template <int kStride, bool kAsym, int kFast>
__global__ void __launch_bounds__(kDwThreads, 2)
depthwise3x3_kernel(const __grid_constant__ CUtensorMap map_x, const DwArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base_addr = (smem_u32(smem_raw) + 127u) & ~127u;
    uint8_t* const smem = smem_raw + (base_addr - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bars[2];
    __shared__ int abort_flag;
    const uint32_t bar0 = smem_u32(&bars[0]);

    if (threadIdx.x == 0) {
        mbar_init(bar0, 1);
        mbar_init(bar0 + 8, 1);
        abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&map_x);
    }
    __syncthreads();

    auto issue = [&](int64_t tile, uint32_t buf) {   // thread 0 only
        const TileCoord t = decode_tile(a, tile);
        mbar_arrive_expect_tx(bar0 + 8 * buf, a.tile_bytes);
        tma_load_4d(base_addr + buf * a.buf_stride, &map_x, bar0 + 8 * buf, t.cc * a.cb, t.w0 * kStride - 1,
                    t.h0 * kStride - 1, t.b);
    };
    if (threadIdx.x == 0 && blockIdx.x < a.num_tiles) issue(blockIdx.x, 0);

    // thread mapping inside a tile
    const int tid = threadIdx.x;
    const int g = tid % a.gp;
    const int pr = (tid / a.gp) % a.pairs;
    const int sl = tid / (a.gp * a.pairs);
    const bool in_slot = sl < a.slots;
    const int r_begin = sl * a.rps;

    uint32_t w1[3][8];
    Requant rq;
    int32_t base[8];
    rq.zy = a.zy;
    rq.lo = a.act_min;
    rq.span = a.act_max - a.act_min;
    rq.lo4 = 0x01010101u * static_cast<uint32_t>(a.act_min);
    const uint32_t fill = 0x01010101u * static_cast<uint32_t>(a.zx);
    int loaded_cc = -1;

    uint32_t it = 0;
    for (int64_t tile = blockIdx.x; tile < a.num_tiles; tile += gridDim.x, ++it) {
        const uint32_t buf = it & 1, parity = (it >> 1) & 1;
        const TileCoord t = decode_tile(a, tile);
        // prefetch the next tile into the other buffer (its previous use ended at the last __syncthreads)
        if (threadIdx.x == 0 && tile + gridDim.x < a.num_tiles) {
            fence_proxy_async_smem();   // border cells written by threads must not overtake the refill
            issue(tile + gridDim.x, buf ^ 1);
        }

        const int c0 = t.cc * a.cb + 8 * g;
        const bool worker = in_slot && c0 < a.c;   // groups entirely beyond the last channel idle
        if (worker && t.cc != loaded_cc) {         // per-channel constants of this channel chunk
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                const uint4 lo = __ldg(reinterpret_cast<const uint4*>(a.taps + static_cast<int64_t>(i) * a.tap_pitch + c0));
                const uint4 hi = __ldg(reinterpret_cast<const uint4*>(a.taps + static_cast<int64_t>(i) * a.tap_pitch + c0 + 4));
                w1[i][0] = lo.x; w1[i][1] = lo.y; w1[i][2] = lo.z; w1[i][3] = lo.w;
                w1[i][4] = hi.x; w1[i][5] = hi.y; w1[i][6] = hi.z; w1[i][7] = hi.w;
            }
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                const int32_t r = a.y_raw ? 40 : __ldg(a.rshift + c0 + ch);   // raw output has no multipliers
                rq.m[ch] = a.y_raw ? 0 : __ldg(a.mult + c0 + ch);
                rq.sh[ch] = kFast != 0 ? r - 32 : r;
                if (kFast == 1) rq.addhi[ch] = (2 * (a.zy - a.act_min) + 1) * (1 << (r - 33));
                if (kFast == 2) rq.add[ch] = static_cast<int64_t>(2 * (a.zy - a.act_min) + 1) << (r - 1);
                base[ch] = __ldg(a.bias + c0 + ch) - a.zx * __ldg(a.wsum + c0 + ch) + 9 * a.zx * a.zw;
            }
            loaded_cc = t.cc;
        }

        if (!mbar_wait(bar0 + 8 * buf, parity, a.wait_budget)) {
            if (atomicCAS(a.status, 0, QTZ_ERR_DEVICE_TIMEOUT) == 0) a.status[1] = QTZ_SITE_TMA_FULL;
            abort_flag = 1;
        }
        __syncthreads();
        if (abort_flag) break;

        uint8_t* const tile_s = smem + buf * a.buf_stride;
        // padding is real zero = code z_x: overwrite the cells TMA zero-filled outside the image
        const int ih0 = t.h0 * kStride - 1, iw0 = t.w0 * kStride - 1;
        if (a.zx != 0 && (ih0 < 0 || iw0 < 0 || ih0 + a.thin > a.h || iw0 + a.twin > a.w_)) {
            const int row_bytes = a.twin * a.cb;
            const int rows_in = min(a.thin, a.h - ih0);        // tile rows [first_row, rows_in) are inside the image
            const int first_row = ih0 < 0 ? 1 : 0;
            if (first_row)                                      // the row above the image
                for (int i = 8 * tid; i < row_bytes; i += 8 * kDwThreads) *reinterpret_cast<uint2*>(tile_s + i) = make_uint2(fill, fill);
            for (int ri = rows_in; ri < a.thin; ++ri)           // rows below the image
                for (int i = 8 * tid; i < row_bytes; i += 8 * kDwThreads)
                    *reinterpret_cast<uint2*>(tile_s + ri * row_bytes + i) = make_uint2(fill, fill);
            const int cols_in = min(a.twin, a.w_ - iw0);        // tile columns [first_col, cols_in) are inside
            const int first_col = iw0 < 0 ? 1 : 0;
            if (first_col + a.twin - cols_in > 0) {             // the left column and / or the right columns
                const int lane8 = 8 * (tid & 31), warp_id = tid >> 5;
                for (int ri = first_row + warp_id; ri < rows_in; ri += kDwThreads / 32) {
                    uint8_t* row = tile_s + ri * row_bytes;
                    if (first_col)
                        for (int i = lane8; i < a.cb; i += 256) *reinterpret_cast<uint2*>(row + i) = make_uint2(fill, fill);
                    for (int i = lane8; i < (a.twin - cols_in) * a.cb; i += 256)
                        *reinterpret_cast<uint2*>(row + cols_in * a.cb + i) = make_uint2(fill, fill);
                }
            }
            __syncthreads();
        }

        const int ow0 = t.w0 + 2 * pr;
        if (worker && ow0 < a.ow) {
            const int r_end = min(min(a.th, r_begin + a.rps), a.oh - t.h0);   // tile-local output rows of this thread
            const uint8_t* cell = tile_s + (r_begin * kStride * a.twin + 2 * pr * kStride) * a.cb + 8 * g;
            const int row_bytes = a.twin * a.cb;
            const int64_t first_px = (static_cast<int64_t>(t.b) * a.oh + t.h0 + r_begin) * a.ow + ow0;
            uint8_t* out = a.y + first_px * a.yp + c0;
            int32_t* out_raw = a.y_raw + first_px * a.c + c0;
            const int64_t out_row = static_cast<int64_t>(a.ow) * a.yp;
            const bool second = ow0 + 1 < a.ow;

            auto finish = [&](int32_t (&acc)[2][8], int32_t (&xs)[2][8]) {
                int32_t v[8];
                if (a.y_raw) {   // calibration: the accumulators themselves
#pragma unroll
                    for (int j = 0; j < 2; ++j)
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch)
                            if ((j == 0 || second) && c0 + ch < a.c)
                                out_raw[j * a.c + ch] = acc[j][ch] - (kAsym ? a.zw * xs[j][ch] : 0);
                    out_raw += static_cast<int64_t>(a.ow) * a.c;
                    return;
                }
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) v[ch] = acc[0][ch] - (kAsym ? a.zw * xs[0][ch] : 0);
                *reinterpret_cast<uint2*>(out) = requant_pixel<kFast>(v, rq);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) v[ch] = acc[1][ch] - (kAsym ? a.zw * xs[1][ch] : 0);
                const uint2 o1 = requant_pixel<kFast>(v, rq);
                if (second) *reinterpret_cast<uint2*>(out + a.yp) = o1;
                out += out_row;
            };

            int32_t acc[2][8], xs[2][8];
            if (kStride == 1) {
                // three input rows stay in registers and rotate: tile rows r, r+1, r+2 feed output row r
                RowState<1> r0, r1, r2;
                load_row<1>(cell, a.cb, r0); cell += row_bytes;
                load_row<1>(cell, a.cb, r1); cell += row_bytes;
                for (int r = r_begin; r < r_end; r += 3) {
                    load_row<1>(cell, a.cb, r2); cell += row_bytes;
                    mac_row<1, kAsym, true>(r0, w1[0], base, acc, xs); mac_row<1, kAsym, false>(r1, w1[1], base, acc, xs);
                    mac_row<1, kAsym, false>(r2, w1[2], base, acc, xs);
                    finish(acc, xs);
                    if (r + 1 >= r_end) break;
                    load_row<1>(cell, a.cb, r0); cell += row_bytes;
                    mac_row<1, kAsym, true>(r1, w1[0], base, acc, xs); mac_row<1, kAsym, false>(r2, w1[1], base, acc, xs);
                    mac_row<1, kAsym, false>(r0, w1[2], base, acc, xs);
                    finish(acc, xs);
                    if (r + 2 >= r_end) break;
                    load_row<1>(cell, a.cb, r1); cell += row_bytes;
                    mac_row<1, kAsym, true>(r2, w1[0], base, acc, xs); mac_row<1, kAsym, false>(r0, w1[1], base, acc, xs);
                    mac_row<1, kAsym, false>(r1, w1[2], base, acc, xs);
                    finish(acc, xs);
                }
            } else {
                // stride 2: tile rows 2r, 2r+1, 2r+2; the last one is the next output row's first
                RowState<2> top, mid, bot;
                load_row<2>(cell, a.cb, top); cell += row_bytes;
                for (int r = r_begin; r < r_end; r += 2) {
                    load_row<2>(cell, a.cb, mid); cell += row_bytes;
                    load_row<2>(cell, a.cb, bot); cell += row_bytes;
                    mac_row<2, kAsym, true>(top, w1[0], base, acc, xs); mac_row<2, kAsym, false>(mid, w1[1], base, acc, xs);
                    mac_row<2, kAsym, false>(bot, w1[2], base, acc, xs);
                    finish(acc, xs);
                    if (r + 1 >= r_end) break;
                    load_row<2>(cell, a.cb, mid); cell += row_bytes;
                    load_row<2>(cell, a.cb, top); cell += row_bytes;
                    mac_row<2, kAsym, true>(bot, w1[0], base, acc, xs); mac_row<2, kAsym, false>(mid, w1[1], base, acc, xs);
                    mac_row<2, kAsym, false>(top, w1[2], base, acc, xs);
                    finish(acc, xs);
                }
            }
        }
        __syncthreads();   // everyone is done with this buffer before it is refilled two tiles later
    }
}

template <int kStride, bool kAsym>
void launch_variant(int fast, unsigned blocks, size_t smem, cudaStream_t st, const CUtensorMap& map, const DwArgs& a)
{
    if (fast == 1)
        depthwise3x3_kernel<kStride, kAsym, 1><<<blocks, kDwThreads, smem, st>>>(map, a);
    else if (fast == 2)
        depthwise3x3_kernel<kStride, kAsym, 2><<<blocks, kDwThreads, smem, st>>>(map, a);
    else
        depthwise3x3_kernel<kStride, kAsym, 0><<<blocks, kDwThreads, smem, st>>>(map, a);
}

template <int kStride, bool kAsym>
cudaError_t allow_smem()
{
    cudaError_t e = cudaFuncSetAttribute(depthwise3x3_kernel<kStride, kAsym, 0>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemLimit);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(depthwise3x3_kernel<kStride, kAsym, 1>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemLimit);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(depthwise3x3_kernel<kStride, kAsym, 2>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemLimit);
    return e;
}

}  // namespace

struct qtz_dw_state {
    DwArgs args{};
    uint32_t smem_bytes = 0;
    int grid = 0;
};

// Chooses the tile (channel chunk, output columns and rows) and the thread mapping.
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
    a.gp = a.cb / 8;
    // columns: as many pairs as fit the block and the image, split evenly over the tiles of a row
    const int all_pairs = (p->ow + 1) / 2;
    const int max_pairs = std::max(1, std::min(kDwThreads / a.gp, all_pairs));
    const int tiles_w = (all_pairs + max_pairs - 1) / max_pairs;
    a.pairs = (all_pairs + tiles_w - 1) / tiles_w;
    a.tw = 2 * a.pairs;
    a.twin = (a.tw - 1) * st + 3;
    a.slots = std::max(1, kDwThreads / (a.gp * a.pairs));
    // rows: about 40 KB per buffer
    const int thin_max = std::max(3, 40 * 1024 / (a.twin * a.cb));
    int th = std::min(std::max(1, (thin_max - 3) / st + 1), p->oh);
    a.tiles_h = (p->oh + th - 1) / th;
    th = (p->oh + a.tiles_h - 1) / a.tiles_h;
    a.slots = std::min(a.slots, th);
    a.rps = (th + a.slots - 1) / a.slots;
    a.th = th;
    a.thin = (a.th - 1) * st + 3;
    if (a.twin > 256 || a.thin > 256) return QTZ_ERR_UNSUPPORTED;
    a.tiles_w = (p->ow + a.tw - 1) / a.tw;
    a.num_tiles = static_cast<int64_t>(a.c_chunks) * d.batch * a.tiles_h * a.tiles_w;
    a.tile_bytes = static_cast<uint32_t>(a.thin) * a.twin * a.cb;
    a.buf_stride = (a.tile_bytes + 127u) & ~127u;
    s->smem_bytes = 2 * a.buf_stride + 128;
    if (s->smem_bytes > static_cast<uint32_t>(kDwSmemLimit)) return QTZ_ERR_UNSUPPORTED;
    const int per_sm = std::max(1, std::min(2, static_cast<int>((220 * 1024) / (s->smem_bytes + 1024))));
    s->grid = static_cast<int>(std::min<int64_t>(a.num_tiles, static_cast<int64_t>(p->h->num_sms) * per_sm));
    a.taps = p->dw_taps; a.wsum = p->dw_wsum; a.bias = p->bias; a.mult = p->mult; a.rshift = p->rshift;
    a.status = p->h->status_dev;
    a.wait_budget = 2000000000LL;
    a.zw = p->w_zp_signed;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = allow_smem<1, false>();
        if (e == cudaSuccess) e = allow_smem<1, true>();
        if (e == cudaSuccess) e = allow_smem<2, false>();
        if (e == cudaSuccess) e = allow_smem<2, true>();
        if (e != cudaSuccess) return qtz_cuda_fail(p->h, e, "cudaFuncSetAttribute(depthwise3x3_kernel)");
        attr_set = true;
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
    CUtensorMap map;
    const uint64_t pitch = static_cast<uint64_t>(d.c_pitch_in);
    const uint64_t dims[4] = {static_cast<uint64_t>(d.c), static_cast<uint64_t>(d.w), static_cast<uint64_t>(d.h),
                              static_cast<uint64_t>(d.batch)};
    const uint64_t strides[3] = {pitch, pitch * d.w, pitch * d.w * d.h};
    const uint32_t box[4] = {static_cast<uint32_t>(a.cb), static_cast<uint32_t>(a.twin), static_cast<uint32_t>(a.thin), 1u};
    if (!qtz_encode_u8_map(&map, x, 4, dims, strides, box, 0)) {
        p->h->last_error = "cuTensorMapEncodeTiled failed for the depthwise input";
        return QTZ_ERR_CUDA;
    }
    // requantisation form: 1 for right shifts 33..53, 2 for 32..53 (64-bit rounding constant), 0 for any shift
    const int fast = (raw || p->rshift_max > 53 || p->rshift_min < 32) ? 0 : (p->rshift_min >= 33 ? 1 : 2);
    const bool asym = p->w_zp_signed != 0;
    if (p->ev_start) QTZ_CUDA(p->h, cudaEventRecord(p->ev_start, st));
    const unsigned blocks = static_cast<unsigned>(p->dw->grid);
    if (d.stride == 1) {
        if (asym) launch_variant<1, true>(fast, blocks, p->dw->smem_bytes, st, map, a);
        else launch_variant<1, false>(fast, blocks, p->dw->smem_bytes, st, map, a);
    } else {
        if (asym) launch_variant<2, true>(fast, blocks, p->dw->smem_bytes, st, map, a);
        else launch_variant<2, false>(fast, blocks, p->dw->smem_bytes, st, map, a);
    }
    QTZ_LAUNCH_CHECK(p->h, "depthwise3x3_kernel");
    if (p->ev_stop) QTZ_CUDA(p->h, cudaEventRecord(p->ev_stop, st));
    return QTZ_OK;
}
