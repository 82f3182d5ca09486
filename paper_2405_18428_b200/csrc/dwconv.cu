// SREM depthwise 3x3 convolution (Algorithm 1: DWConv2d on the reshaped token matrix), channel-last.
// A CTA stages a (TY+2) x (TX+2) pixel halo tile of CH channels in shared memory with 16-byte
// coalesced loads; each thread then owns 8 channels of one tile column and walks down the rows.
// The scan order the residual stream is in (`dir`) only permutes the filter taps:
// reverse orders see the filter rotated by 180 degrees, column orders see it transposed.
#include <type_traits>

#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int TY = 4, TX = 8, VEC = 8;
// Channels per CTA: 256 bytes of one pixel, so the halo tile stays under 48 KB of shared memory.
template <typename T> struct Cfg {
    static constexpr int CH = 256 / (int)sizeof(T);
    static constexpr int kLanes = CH / VEC;          // 16-byte (bf16) / 32-byte (fp32) vectors per pixel
    static constexpr int kThreads = kLanes * TX;
};

template <typename T> struct Vec8;
template <> struct Vec8<float> {
    float4 a, b;
    __device__ static Vec8 load(const float *p) { return {load4(p), load4(p + 4)}; }
    __device__ static Vec8 zero() { return {make_float4(0, 0, 0, 0), make_float4(0, 0, 0, 0)}; }
    __device__ void unpack(float (&f)[8]) const { f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w; }
};
template <> struct Vec8<__nv_bfloat16> {
    uint4 u;
    __device__ static Vec8 load(const __nv_bfloat16 *p) { return {*reinterpret_cast<const uint4 *>(p)}; }
    __device__ static Vec8 zero() { return {make_uint4(0, 0, 0, 0)}; }
    __device__ void unpack(float (&f)[8]) const
    {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

__device__ __forceinline__ void store8(float *p, const float (&f)[8])
{
    store4(p, make_float4(f[0], f[1], f[2], f[3]));
    store4(p + 4, make_float4(f[4], f[5], f[6], f[7]));
}
__device__ __forceinline__ void store8(__nv_bfloat16 *p, const float (&f)[8])
{
    uint4 u;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(f[0], f[1]); u.x = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[2], f[3]); u.y = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[4], f[5]); u.z = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[6], f[7]); u.w = *reinterpret_cast<uint32_t *>(&t);
    *reinterpret_cast<uint4 *>(p) = u;
}

template <typename T, typename TO>
__global__ void __launch_bounds__(Cfg<T>::kThreads)
srem_dwconv3x3(const T *__restrict__ x, const T *__restrict__ w, const T *__restrict__ bias,
               TO *__restrict__ y, int gh, int gw, int D, int nchb, int dir)
{
    constexpr int CH = Cfg<T>::CH, kLanes = Cfg<T>::kLanes, kConvThreads = Cfg<T>::kThreads;
    __shared__ Vec8<T> tile[TY + 2][TX + 2][kLanes];
    const int b = blockIdx.z / nchb, chb = blockIdx.z - b * nchb;
    const int x0 = blockIdx.x * TX, y0 = blockIdx.y * TY;
    const int lane = threadIdx.x % kLanes, col = threadIdx.x / kLanes;
    const int ch = chb * CH + lane * VEC;
    const bool ch_ok = ch < D;
    const T *xb = x + (size_t)b * gh * gw * D;
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed

    for (int idx = threadIdx.x; idx < (TY + 2) * (TX + 2) * kLanes; idx += kConvThreads) {
        const int l = idx % kLanes, pix = idx / kLanes;
        const int tx = pix % (TX + 2), ty = pix / (TX + 2);
        const int gy = y0 + ty - 1, gx = x0 + tx - 1, c = chb * CH + l * VEC;
        Vec8<T> v = Vec8<T>::zero();
        if (gy >= 0 && gy < gh && gx >= 0 && gx < gw && c < D)
            v = Vec8<T>::load(xb + ((size_t)gy * gw + gx) * D + c);
        tile[ty][tx][l] = v;
    }
    // filter taps for this thread's channels, re-oriented: wt[u][v] multiplies x[i+u-1][j+v-1].  They are
    // kept packed (and unpacked at every use) so that the kernel stays at a register count that lets
    // six CTAs share an SM; the loads of the tile are what it waits for, not the arithmetic.
    Vec8<T> wt[3][3];
    float bs[8];
#pragma unroll
    for (int u = 0; u < 3; ++u)
#pragma unroll
        for (int v = 0; v < 3; ++v) {
            int su = u, sv = v;
            if (dir & 2) { su = v; sv = u; }
            if (dir & 1) { su = 2 - su; sv = 2 - sv; }
            wt[u][v] = ch_ok ? Vec8<T>::load(w + (size_t)(su * 3 + sv) * D + ch) : Vec8<T>::zero();
        }
#pragma unroll
    for (int i = 0; i < 8; ++i) bs[i] = 0.f;
    if (bias != nullptr && ch_ok) Vec8<T>::load(bias + ch).unpack(bs);
    __syncthreads();
    if (!ch_ok || x0 + col >= gw) return;

#pragma unroll
    for (int ty = 0; ty < TY; ++ty) {
        if (y0 + ty < gh) {
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = bs[i];
#pragma unroll
            for (int u = 0; u < 3; ++u)
#pragma unroll
                for (int v = 0; v < 3; ++v) {
                    float xv[8], wv[8];
                    tile[ty + u][col + v][lane].unpack(xv);
                    wt[u][v].unpack(wv);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[i] = fmaf(wv[i], xv[i], acc[i]);
                }
            store8(y + (((size_t)b * gh + y0 + ty) * gw + x0 + col) * D + ch, acc);
        }
    }
}

// The same convolution for grids that fill the machine: a CTA walks down a strip of TX pixel columns and
// CH channels, row by row.  Input rows (TX + 2 pixels with the halo) arrive through cp.async in a ring of
// kRing rows, kRing - 1 rows ahead of the arithmetic, so every input row is fetched once per strip.  A thread
// owns 4 channels of two neighbouring pixel columns: it widens the four pixels around them once per row and
// feeds the three output rows around that row from registers (acc[r % 3] belongs to output row r); at this
// register count four CTAs share an SM.  Out-of-grid pixels and channels are zero-filled by the copy itself (source size 0).  One barrier
// per row: the slot refilled after the barrier of row r is the one row r - 1 was read from.
// Strip s = ((channel block * B + batch) * strips_x + strip column) * nseg + row segment; a row segment
// covers seg_rows output rows (plus one halo row on either side).
constexpr int kRing = 6;

template <typename T, typename TO>
__global__ void __launch_bounds__(Cfg<T>::kThreads, 4)
srem_dwconv3x3_strip(const T *__restrict__ x, const T *__restrict__ w, const T *__restrict__ bias,
                     TO *__restrict__ y, int B, int gh, int gw, int D, int dir, int strips_x, int nseg, int seg_rows,
                     int nstrips)
{
    constexpr int CH = Cfg<T>::CH, kLanes = Cfg<T>::kLanes, kConvThreads = Cfg<T>::kThreads;
    constexpr int kPieces = (int)sizeof(Vec8<T>) / 16;
    constexpr int kRowVecs = (TX + 2) * kLanes;                  // 16/32-byte vectors of one input row of the strip
    constexpr int kFill = (kRowVecs + kConvThreads - 1) / kConvThreads;
    constexpr int kQuads = CH / 4;                                // 4-channel groups of a pixel
    static_assert(kQuads * (TX / 2) == kConvThreads, "one thread per (column pair, channel quad)");
    __shared__ Vec8<T> ring[kRing][TX + 2][kLanes];
    const int quad = threadIdx.x % kQuads, c0 = 2 * (threadIdx.x / kQuads);     // first of the thread's two columns
    pdl_wait();
    pdl_launch_dependents();
    int cur_chb = -1;
    float wf[3][3][4], bs[4];
    for (int s = blockIdx.x; s < nstrips; s += gridDim.x) {
        const int sg = s % nseg, s1 = s / nseg, sx = s1 % strips_x, s2 = s1 / strips_x, b = s2 % B, chb = s2 / B;
        const int x0 = sx * TX, ys = sg * seg_rows, ye = min(ys + seg_rows, gh), nr = ye - ys + 2;
        const int ch = chb * CH + quad * 4;
        const bool ch_ok = ch < D, ok0 = ch_ok && x0 + c0 < gw, ok1 = ch_ok && x0 + c0 + 1 < gw;
        const T *xb = x + (size_t)b * gh * gw * D;
        // this thread's vectors of an input row: pixel column, validity and offsets stay the same for every row
        int f_off[kFill];
        uint32_t f_dst[kFill];
        bool f_ok[kFill];
#pragma unroll
        for (int i = 0; i < kFill; ++i) {
            const int idx = (int)threadIdx.x + i * kConvThreads, l = idx % kLanes, tx = idx / kLanes;
            const int gx = x0 + tx - 1, c = chb * CH + l * VEC;
            f_ok[i] = idx < kRowVecs && gx >= 0 && gx < gw && c < D;
            f_off[i] = f_ok[i] ? gx * D + c : 0;
            f_dst[i] = idx < kRowVecs ? (uint32_t)__cvta_generic_to_shared(&ring[0][tx][l]) : 0u;
        }
        auto fill = [&](int rr) {       // input row rr of the strip (image row ys - 1 + rr) into its ring slot
            const int gy = ys - 1 + rr;
            const bool row_ok = gy >= 0 && gy < gh;
            const T *row = xb + (size_t)(row_ok ? gy : 0) * gw * D;
            const uint32_t slot = (uint32_t)(rr % kRing) * (uint32_t)sizeof(ring[0]);
#pragma unroll
            for (int i = 0; i < kFill; ++i) {
                if (i + 1 < kFill || (int)threadIdx.x + i * kConvThreads < kRowVecs) {
                    const bool in = row_ok && f_ok[i];
                    const char *src = reinterpret_cast<const char *>(in ? row + f_off[i] : x);
#pragma unroll
                    for (int p = 0; p < kPieces; ++p)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(f_dst[i] + slot + 16 * p),
                                     "l"(src + (in ? 16 * p : 0)), "r"(in ? 16 : 0) : "memory");
                }
            }
        };
        __syncthreads();                // the previous strip's last rows have been read
#pragma unroll
        for (int i = 0; i < kRing - 1; ++i) {
            if (i < nr) fill(i);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        if (chb != cur_chb) {            // uniform over the CTA: the taps of this channel block, re-oriented
            cur_chb = chb;
#pragma unroll
            for (int u = 0; u < 3; ++u)
#pragma unroll
                for (int v = 0; v < 3; ++v) {
                    int su = u, sv = v;
                    if (dir & 2) { su = v; sv = u; }
                    if (dir & 1) { su = 2 - su; sv = 2 - sv; }
                    const float4 t = ch_ok ? load4(w + (size_t)(su * 3 + sv) * D + ch) : make_float4(0.f, 0.f, 0.f, 0.f);
                    wf[u][v][0] = t.x; wf[u][v][1] = t.y; wf[u][v][2] = t.z; wf[u][v][3] = t.w;
                }
            const float4 t = (bias != nullptr && ch_ok) ? load4(bias + ch) : make_float4(0.f, 0.f, 0.f, 0.f);
            bs[0] = t.x; bs[1] = t.y; bs[2] = t.z; bs[3] = t.w;
        }
        float acc[3][2][4];
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[r][0][i] = acc[r][1][i] = 0.f;
        TO *yrow = y + (((size_t)b * gh + ys) * gw + x0 + c0) * D + ch;      // output row completed next
        // One input row: PH = rr % 3 is a compile-time constant so that the accumulators stay in registers.
        // Row rr starts output row rr (of the segment), feeds rr - 1 and completes rr - 2.  The rows before the
        // first and after the last output row accumulate into registers that are re-initialised or dropped.
        auto step = [&](int rr, auto ph_tag) {
            constexpr int PH = decltype(ph_tag)::value;
            asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 2) : "memory");      // row rr has landed
            __syncthreads();
            if (rr + kRing - 1 < nr) fill(rr + kRing - 1);
            asm volatile("cp.async.commit_group;" ::: "memory");
            float xv[4][4];
            const T *rowp = reinterpret_cast<const T *>(&ring[rr % kRing][0][0]) + quad * 4;     // [TX + 2][CH] elements
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const float4 t = load4(rowp + (c0 + v) * CH);
                xv[v][0] = t.x; xv[v][1] = t.y; xv[v][2] = t.z; xv[v][3] = t.w;
            }
#pragma unroll
            for (int p = 0; p < 2; ++p)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[PH][p][i] = bs[i];
#pragma unroll
            for (int u = 0; u < 3; ++u)
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int v = 0; v < 3; ++v)
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float &a = acc[(PH + 3 - u) % 3][p][i];
                            a = fmaf(wf[u][v][i], xv[p + v][i], a);
                        }
            if (rr >= 2) {
                const float (&r0)[4] = acc[(PH + 1) % 3][0], (&r1)[4] = acc[(PH + 1) % 3][1];
                if (ok0) store4(yrow, make_float4(r0[0], r0[1], r0[2], r0[3]));
                if (ok1) store4(yrow + D, make_float4(r1[0], r1[1], r1[2], r1[3]));
                yrow += (size_t)gw * D;
            }
        };
        for (int rr = 0; rr < nr; rr += 3) {
            step(rr, std::integral_constant<int, 0>{});
            if (rr + 1 < nr) step(rr + 1, std::integral_constant<int, 1>{});
            if (rr + 2 < nr) step(rr + 2, std::integral_constant<int, 2>{});
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ---- reverse mode: filter and bias gradients ------------------------------------------------------
// dw'[u][v][c] = sum over pixels of dy[i][j][c] * x[i+u-1][j+v-1][c] (zero outside the grid), computed
// in canonical taps and written to the stored tap the scan order maps (u, v) to; dbias = sum of dy.
// Same walk as the forward strip kernel: a CTA goes down strips of TX pixel columns and CH channels row
// by row, rows of x (with the halo) and of dy arriving through cp.async rings.  A thread owns 4 channels
// of two neighbouring columns: input row r meets the dy rows r, r - 1, r - 2 (kept in registers, g[r % 3]
// is dy row r) in the taps u = 0, 1, 2 and adds 72 products to its 36 + 4 accumulators.  CTA y of a
// channel block takes the strips y, y + gridDim.y, ... in that order; then the CTA's column pairs are
// summed through shared memory and one partial sum per CTA is written; a second kernel adds the partial
// sums in a fixed order, so the result does not depend on scheduling.  The dy rows a CTA reads are those
// of its own row segment only (segments share halo rows of x, not output rows).
constexpr int kWgPixels = 128;       // pixels per partial sum (sizes the workspace)

template <typename T>
__global__ void __launch_bounds__(Cfg<T>::kThreads, 4)
srem_dwconv_wgrad(const T *__restrict__ x, const T *__restrict__ dy, float *__restrict__ partial,
                  int B, int gh, int gw, int D, int dir, int strips_x, int nseg, int seg_rows, int nstrips)
{
    constexpr int CH = Cfg<T>::CH, kLanes = Cfg<T>::kLanes, kConvThreads = Cfg<T>::kThreads;
    constexpr int kPieces = (int)sizeof(Vec8<T>) / 16, kQuads = CH / 4, kWarps = kConvThreads / 32;
    constexpr int kRowX = (TX + 2) * kLanes, kRowG = TX * kLanes, kRowVecs = kRowX + kRowG;
    constexpr int kFill = (kRowVecs + kConvThreads - 1) / kConvThreads;
    // rings of x rows and dy rows; the same memory later holds the per-warp sums [warps][10][CH]
    constexpr size_t kRingBytes = sizeof(Vec8<T>) * kRing * kRowVecs, kRedBytes = sizeof(float) * kWarps * 10 * CH;
    __shared__ __align__(16) char sm[kRingBytes > kRedBytes ? kRingBytes : kRedBytes];
    Vec8<T> (*xring)[TX + 2][kLanes] = reinterpret_cast<Vec8<T> (*)[TX + 2][kLanes]>(sm);
    Vec8<T> (*gring)[TX][kLanes] = reinterpret_cast<Vec8<T> (*)[TX][kLanes]>(sm + sizeof(Vec8<T>) * kRing * kRowX);
    const int quad = threadIdx.x % kQuads, c0 = 2 * (threadIdx.x / kQuads);
    const int chb = blockIdx.x;
    pdl_wait();
    pdl_launch_dependents();
    float acc[3][3][4], accb[4];
#pragma unroll
    for (int u = 0; u < 3; ++u)
#pragma unroll
        for (int v = 0; v < 3; ++v)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[u][v][i] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) accb[i] = 0.f;
    for (int s = blockIdx.y; s < nstrips; s += gridDim.y) {
        const int sg = s % nseg, s1 = s / nseg, sx = s1 % strips_x, b = s1 / strips_x;
        const int x0 = sx * TX, ys = sg * seg_rows, ye = min(ys + seg_rows, gh), nr = ye - ys + 2;
        const T *xb = x + (size_t)b * gh * gw * D, *gb = dy + (size_t)b * gh * gw * D;
        // this thread's vectors of a row pair (x row with halo, then dy row): columns and offsets stay the same
        int f_off[kFill];
        uint32_t f_dst[kFill];
        bool f_ok[kFill], f_isx[kFill];
#pragma unroll
        for (int i = 0; i < kFill; ++i) {
            const int idx = (int)threadIdx.x + i * kConvThreads;
            const bool isx = idx < kRowX;
            const int j = isx ? idx : idx - kRowX, l = j % kLanes, tx = j / kLanes;
            const int gx = isx ? x0 + tx - 1 : x0 + tx, c = chb * CH + l * VEC;
            f_isx[i] = isx;
            f_ok[i] = idx < kRowVecs && gx >= 0 && gx < gw && c < D;
            f_off[i] = f_ok[i] ? gx * D + c : 0;
            f_dst[i] = idx >= kRowVecs ? 0u
                       : isx ? (uint32_t)__cvta_generic_to_shared(&xring[0][tx][l]) : (uint32_t)__cvta_generic_to_shared(&gring[0][tx][l]);
        }
        auto fill = [&](int rr) {       // x row rr of the strip (image row ys - 1 + rr) and dy row rr (image row ys + rr)
            const int gyx = ys - 1 + rr, gyg = ys + rr;
            const bool okx = gyx >= 0 && gyx < gh, okg = gyg < ye;
            const T *rowx = xb + (size_t)(okx ? gyx : 0) * gw * D, *rowg = gb + (size_t)(okg ? gyg : 0) * gw * D;
            const uint32_t slx = (uint32_t)(rr % kRing) * (uint32_t)sizeof(xring[0]), slg = (uint32_t)(rr % kRing) * (uint32_t)sizeof(gring[0]);
#pragma unroll
            for (int i = 0; i < kFill; ++i) {
                if (i + 1 < kFill || (int)threadIdx.x + i * kConvThreads < kRowVecs) {
                    const bool in = f_ok[i] && (f_isx[i] ? okx : okg);
                    const char *src = reinterpret_cast<const char *>(in ? (f_isx[i] ? rowx : rowg) + f_off[i] : x);
                    const uint32_t dst = f_dst[i] + (f_isx[i] ? slx : slg);
#pragma unroll
                    for (int p = 0; p < kPieces; ++p)
                        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst + 16 * p), "l"(src + (in ? 16 * p : 0)),
                                     "r"(in ? 16 : 0) : "memory");
                }
            }
        };
        __syncthreads();                // the previous strip's last rows have been read
#pragma unroll
        for (int i = 0; i < kRing - 1; ++i) {
            if (i < nr) fill(i);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        float g[3][2][4];
#pragma unroll
        for (int r = 0; r < 3; ++r)
#pragma unroll
            for (int i = 0; i < 4; ++i) g[r][0][i] = g[r][1][i] = 0.f;
        // One row: PH = rr % 3 is a compile-time constant so that the dy rows stay in registers.
        auto step = [&](int rr, auto ph_tag) {
            constexpr int PH = decltype(ph_tag)::value;
            asm volatile("cp.async.wait_group %0;" ::"n"(kRing - 2) : "memory");      // rows rr have landed
            __syncthreads();
            if (rr + kRing - 1 < nr) fill(rr + kRing - 1);
            asm volatile("cp.async.commit_group;" ::: "memory");
            float xv[4][4];
            const T *rowp = reinterpret_cast<const T *>(&xring[rr % kRing][0][0]) + quad * 4;
            const T *rowg = reinterpret_cast<const T *>(&gring[rr % kRing][0][0]) + quad * 4;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                const float4 t = load4(rowp + (c0 + v) * CH);
                xv[v][0] = t.x; xv[v][1] = t.y; xv[v][2] = t.z; xv[v][3] = t.w;
            }
#pragma unroll
            for (int p = 0; p < 2; ++p) {
                const float4 t = load4(rowg + (c0 + p) * CH);       // zero past the segment's last row and past the grid
                g[PH][p][0] = t.x; g[PH][p][1] = t.y; g[PH][p][2] = t.z; g[PH][p][3] = t.w;
#pragma unroll
                for (int i = 0; i < 4; ++i) accb[i] += g[PH][p][i];
            }
#pragma unroll
            for (int u = 0; u < 3; ++u)
#pragma unroll
                for (int p = 0; p < 2; ++p)
#pragma unroll
                    for (int v = 0; v < 3; ++v)
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            acc[u][v][i] = fmaf(g[(PH + 3 - u) % 3][p][i], xv[p + v][i], acc[u][v][i]);
        };
        for (int rr = 0; rr < nr; rr += 3) {
            step(rr, std::integral_constant<int, 0>{});
            if (rr + 1 < nr) step(rr + 1, std::integral_constant<int, 1>{});
            if (rr + 2 < nr) step(rr + 2, std::integral_constant<int, 2>{});
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    // sum over the column pairs: those a warp holds by shuffles (a warp is 32 / kQuads column pairs of all
    // quads), the warps through shared memory
    float *red = reinterpret_cast<float *>(sm);
    const int warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < 10; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float v = k < 9 ? acc[k / 3][k % 3][e] : accb[e];
#pragma unroll
            for (int m = kQuads; m < 32; m <<= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
            if ((threadIdx.x & 31) < kQuads) red[(warp * 10 + k) * CH + quad * 4 + e] = v;
        }
    __syncthreads();
    // partial[part][k][D]: k = stored tap index 0..8, 9 = bias
    for (int idx = threadIdx.x; idx < 10 * CH; idx += kConvThreads) {
        const int k = idx / CH, c = idx - k * CH;
        if (blockIdx.x * CH + c >= D) continue;
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < kWarps; ++j) sum += red[(j * 10 + k) * CH + c];
        int ks = k;
        if (k < 9) {
            int su = k / 3, sv = k - 3 * su;
            if (dir & 2) { const int tt = su; su = sv; sv = tt; }
            if (dir & 1) { su = 2 - su; sv = 2 - sv; }
            ks = su * 3 + sv;
        }
        partial[((size_t)blockIdx.y * 10 + ks) * D + blockIdx.x * CH + c] = sum;
    }
}

// One warp per output value: its lanes add every 32nd partial sum, then a butterfly (a fixed order).
__global__ void __launch_bounds__(256)
srem_dwconv_wgrad_sum(const float *__restrict__ partial, float *__restrict__ dw, float *__restrict__ dbias,
                      int nslab, int D)
{
    pdl_wait();
    pdl_launch_dependents();
    const int idx = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (idx >= 10 * D) return;          // uniform over the warp
    float sum = 0.f;
    for (int s = lane; s < nslab; s += 32) sum += partial[(size_t)s * 10 * D + idx];
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, k);
    if (lane != 0) return;
    if (idx < 9 * D) dw[idx] = sum;
    else if (dbias != nullptr) dbias[idx - 9 * D] = sum;
}

}  // namespace

dig_status launch_dwconv(const void *x, const void *w, const void *bias, void *y, int B, int gh,
                         int gw, int D, int dir, int dtype, cudaStream_t stream)
{
    const int CH = dtype == DIG_F32 ? Cfg<float>::CH : Cfg<__nv_bfloat16>::CH;
    const int nchb = (D + CH - 1) / CH;
    const dim3 grid((gw + TX - 1) / TX, (gh + TY - 1) / TY, B * nchb);
    if (grid.y > 65535 || (size_t)B * nchb > 65535) return DIG_ERR_UNSUPPORTED;
    KernelTimer t(KID_DWCONV, stream);
    // grids with at least one tile per resident CTA: strips of TX columns walked row by row, cut into row
    // segments so that about four CTAs per SM (what the kernel's register count lets share an SM) have work
    const long long ntiles = (long long)grid.x * grid.y * grid.z;
    const int sms = device_sm_count();
    if (sms <= 0) return DIG_ERR_CUDA;
    const int resident = sms * 4;
    if (ntiles >= resident && ntiles < (1ll << 31)) {
        const long long cols = (long long)grid.x * B * nchb;        // strips before the cut into row segments
        int nseg = (int)(resident / cols);                          // one wave of CTAs where the strips allow it
        if (nseg < 1) nseg = 1;
        if (nseg > (gh + 7) / 8) nseg = (gh + 7) / 8;               // segments of at least 8 rows (two halo rows each)
        const int seg_rows = (gh + nseg - 1) / nseg;
        nseg = (gh + seg_rows - 1) / seg_rows;
        const long long nstrips = cols * nseg;
        if (nstrips >= (1ll << 31)) return DIG_ERR_UNSUPPORTED;
        const dim3 pgrid((unsigned)(nstrips < resident ? nstrips : resident));
        switch (dtype) {
            case DIG_F32:
                launch_pdl(srem_dwconv3x3_strip<float, float>, pgrid, dim3(Cfg<float>::kThreads), 0, stream, (const float *)x,
                           (const float *)w, (const float *)bias, (float *)y, B, gh, gw, D, dir, (int)grid.x, nseg, seg_rows,
                           (int)nstrips);
                break;
            case DIG_BF16:
                launch_pdl(srem_dwconv3x3_strip<__nv_bfloat16, __nv_bfloat16>, pgrid, dim3(Cfg<__nv_bfloat16>::kThreads), 0, stream,
                           (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, (const __nv_bfloat16 *)bias, (__nv_bfloat16 *)y, B, gh,
                           gw, D, dir, (int)grid.x, nseg, seg_rows, (int)nstrips);
                break;
            case DIG_BF16_F32OUT:
                launch_pdl(srem_dwconv3x3_strip<__nv_bfloat16, float>, pgrid, dim3(Cfg<__nv_bfloat16>::kThreads), 0, stream,
                           (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, (const __nv_bfloat16 *)bias, (float *)y, B, gh, gw, D,
                           dir, (int)grid.x, nseg, seg_rows, (int)nstrips);
                break;
            default: return DIG_ERR_INVALID_ARG;
        }
        return cuda_ok(cudaGetLastError());
    }
    switch (dtype) {
        case DIG_F32:
            launch_pdl(srem_dwconv3x3<float, float>, grid, dim3(Cfg<float>::kThreads), 0, stream,
                       (const float *)x, (const float *)w, (const float *)bias, (float *)y, gh, gw, D, nchb, dir);
            break;
        case DIG_BF16:
            launch_pdl(srem_dwconv3x3<__nv_bfloat16, __nv_bfloat16>, grid, dim3(Cfg<__nv_bfloat16>::kThreads), 0, stream,
                       (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, (const __nv_bfloat16 *)bias,
                       (__nv_bfloat16 *)y, gh, gw, D, nchb, dir);
            break;
        case DIG_BF16_F32OUT:
            launch_pdl(srem_dwconv3x3<__nv_bfloat16, float>, grid, dim3(Cfg<__nv_bfloat16>::kThreads), 0, stream,
                       (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)w, (const __nv_bfloat16 *)bias,
                       (float *)y, gh, gw, D, nchb, dir);
            break;
        default: return DIG_ERR_INVALID_ARG;
    }
    return cuda_ok(cudaGetLastError());
}

size_t dwconv_bwd_workspace_bytes(int B, int gh, int gw, int D)
{
    const size_t nslab = ((size_t)B * gh * gw + kWgPixels - 1) / kWgPixels;
    return nslab * 10 * (size_t)D * sizeof(float);
}

// dx = the forward stencil applied to dy with the filter rotated by 180 degrees, which is the forward
// kernel in the opposite scan sense (dir ^ 1); dw, dbias by the two reduction kernels above.
dig_status launch_dwconv_bwd(const void *x, const void *w, const void *dy, void *dx, float *dw, float *dbias,
                             int B, int gh, int gw, int D, int dir, int dtype, float *partial, cudaStream_t stream)
{
    dig_status st = launch_dwconv(dy, w, nullptr, dx, B, gh, gw, D, dir ^ 1, dtype, stream);
    if (st != DIG_OK) return st;
    // One partial sum per CTA row.  No more CTA rows than stay resident together (four CTAs per SM at this
    // kernel's register count) so that their strip loops end together, never more than the workspace holds;
    // strips are cut into row segments until every CTA row has one.
    const int CHb = dtype == DIG_F32 ? Cfg<float>::CH : Cfg<__nv_bfloat16>::CH;
    const int nchb = (D + CHb - 1) / CHb, resident = device_sm_count() * 4;
    if (resident <= 0) return DIG_ERR_CUDA;
    const long long npix = (long long)B * gh * gw;
    long long nslab = (npix + kWgPixels - 1) / kWgPixels;
    const int cap = resident / nchb > 0 ? resident / nchb : 1;
    if (nslab > cap) nslab = cap;
    const int strips_x = (gw + TX - 1) / TX;
    const long long base = (long long)B * strips_x;
    int nseg = (int)(nslab / base);                                 // rounded down: no CTA row gets a second strip while others have one
    if (nseg > (gh + 7) / 8) nseg = (gh + 7) / 8;                   // segments of at least 8 rows
    if (nseg < 1) nseg = 1;
    const int seg_rows = (gh + nseg - 1) / nseg;
    nseg = (gh + seg_rows - 1) / seg_rows;
    const long long nstrips = base * nseg;
    if (nslab > nstrips) nslab = nstrips;
    if (nslab > 65535 || nstrips >= (1ll << 31)) return DIG_ERR_UNSUPPORTED;
    {
        KernelTimer t(KID_DWCONV_WGRAD, stream);
        const dim3 grid(nchb, (unsigned)nslab);
        if (dtype == DIG_F32)
            launch_pdl(srem_dwconv_wgrad<float>, grid, dim3(Cfg<float>::kThreads), 0, stream, (const float *)x, (const float *)dy,
                       partial, B, gh, gw, D, dir, strips_x, nseg, seg_rows, (int)nstrips);
        else
            launch_pdl(srem_dwconv_wgrad<__nv_bfloat16>, grid, dim3(Cfg<__nv_bfloat16>::kThreads), 0, stream,
                       (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)dy, partial, B, gh, gw, D, dir, strips_x, nseg, seg_rows,
                       (int)nstrips);
    }
    if (cudaGetLastError() != cudaSuccess) return DIG_ERR_CUDA;
    KernelTimer t(KID_DWCONV_WGRAD, stream);
    launch_pdl(srem_dwconv_wgrad_sum, dim3((10 * D + 7) / 8), dim3(256), 0, stream, (const float *)partial, dw, dbias,
               (int)nslab, D);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
