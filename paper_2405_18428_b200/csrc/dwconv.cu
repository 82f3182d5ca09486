// SREM depthwise 3x3 convolution (Algorithm 1: DWConv2d on the reshaped token matrix), channel-last.
// A CTA stages a (TY+2) x (TX+2) pixel halo tile of CH channels in shared memory with 16-byte
// coalesced loads; each thread then owns 8 channels of one tile column and walks down the rows.
// The scan order the residual stream is in (`dir`) only permutes the filter taps:
// reverse orders see the filter rotated by 180 degrees, column orders see it transposed.
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

// ---- reverse mode: filter and bias gradients ------------------------------------------------------
// dw'[u][v][c] = sum over pixels of dy[i][j][c] * x[i+u-1][j+v-1][c] (zero outside the grid), computed
// in canonical taps and written to the stored tap the scan order maps (u, v) to; dbias = sum of dy.
// A CTA takes 128 consecutive pixels and one block of channels: its threads (8 channels each, 8
// pixels in flight) read dy and the nine neighbours straight from global memory (they hit L1 / L2),
// reduce over their pixel groups in shared memory and write one partial sum per CTA; a second kernel
// adds the partial sums in a fixed order, so the result does not depend on scheduling.
constexpr int kWgPixels = 128, kWgGroups = 8;

template <typename T>
__global__ void __launch_bounds__(Cfg<T>::kLanes * kWgGroups)
srem_dwconv_wgrad(const T *__restrict__ x, const T *__restrict__ dy, float *__restrict__ partial,
                  int npix, int gh, int gw, int D, int dir)
{
    constexpr int CH = Cfg<T>::CH, kLanes = Cfg<T>::kLanes;
    __shared__ float red[kWgGroups][10][CH];
    const int lane = threadIdx.x % kLanes, grp = threadIdx.x / kLanes;
    const int ch = blockIdx.x * CH + lane * VEC;
    const bool ch_ok = ch < D;
    pdl_wait();
    pdl_launch_dependents();
    float acc[10][8];
#pragma unroll
    for (int k = 0; k < 10; ++k)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[k][i] = 0.f;
    const int p0 = blockIdx.y * kWgPixels, p1 = min(p0 + kWgPixels, npix);
    if (ch_ok) {
        for (int p = p0 + grp; p < p1; p += kWgGroups) {
            const int b = p / (gh * gw), ij = p - b * (gh * gw), i = ij / gw, j = ij - i * gw;
            float g[8];
            Vec8<T>::load(dy + (size_t)p * D + ch).unpack(g);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[9][e] += g[e];
#pragma unroll
            for (int u = 0; u < 3; ++u)
#pragma unroll
                for (int v = 0; v < 3; ++v) {
                    const int ii = i + u - 1, jj = j + v - 1;
                    if (ii < 0 || ii >= gh || jj < 0 || jj >= gw) continue;
                    float xv[8];
                    Vec8<T>::load(x + ((size_t)b * gh * gw + (size_t)ii * gw + jj) * D + ch).unpack(xv);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[u * 3 + v][e] = fmaf(g[e], xv[e], acc[u * 3 + v][e]);
                }
        }
    }
#pragma unroll
    for (int k = 0; k < 10; ++k)
#pragma unroll
        for (int e = 0; e < 8; ++e) red[grp][k][lane * VEC + e] = acc[k][e];
    __syncthreads();
    // partial[slab][k][D]: k = stored tap index 0..8, 9 = bias
    for (int idx = threadIdx.x; idx < 10 * CH; idx += kLanes * kWgGroups) {
        const int k = idx / CH, c = idx - k * CH;
        if (blockIdx.x * CH + c >= D) continue;
        float sum = 0.f;
#pragma unroll
        for (int gidx = 0; gidx < kWgGroups; ++gidx) sum += red[gidx][k][c];
        int ks = k;
        if (k < 9) {
            int su = k / 3, sv = k - 3 * su;
            if (dir & 2) { const int t = su; su = sv; sv = t; }
            if (dir & 1) { su = 2 - su; sv = 2 - sv; }
            ks = su * 3 + sv;
        }
        partial[((size_t)blockIdx.y * 10 + ks) * D + blockIdx.x * CH + c] = sum;
    }
}

__global__ void __launch_bounds__(256)
srem_dwconv_wgrad_sum(const float *__restrict__ partial, float *__restrict__ dw, float *__restrict__ dbias,
                      int nslab, int D)
{
    pdl_wait();
    pdl_launch_dependents();
    const int idx = blockIdx.x * 256 + threadIdx.x;
    if (idx >= 10 * D) return;
    float sum = 0.f;
    for (int s = 0; s < nslab; ++s) sum += partial[(size_t)s * 10 * D + idx];
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
    const int npix = B * gh * gw, nslab = (npix + kWgPixels - 1) / kWgPixels;
    if (nslab > 65535) return DIG_ERR_UNSUPPORTED;
    {
        KernelTimer t(KID_DWCONV_WGRAD, stream);
        if (dtype == DIG_F32) {
            const dim3 grid((D + Cfg<float>::CH - 1) / Cfg<float>::CH, nslab);
            launch_pdl(srem_dwconv_wgrad<float>, grid, dim3(Cfg<float>::kLanes * kWgGroups), 0, stream,
                       (const float *)x, (const float *)dy, partial, npix, gh, gw, D, dir);
        } else {
            const dim3 grid((D + Cfg<__nv_bfloat16>::CH - 1) / Cfg<__nv_bfloat16>::CH, nslab);
            launch_pdl(srem_dwconv_wgrad<__nv_bfloat16>, grid, dim3(Cfg<__nv_bfloat16>::kLanes * kWgGroups), 0, stream,
                       (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)dy, partial, npix, gh, gw, D, dir);
        }
    }
    if (cudaGetLastError() != cudaSuccess) return DIG_ERR_CUDA;
    KernelTimer t(KID_DWCONV_WGRAD, stream);
    launch_pdl(srem_dwconv_wgrad_sum, dim3((10 * D + 255) / 256), dim3(256), 0, stream, (const float *)partial, dw, dbias,
               nslab, D);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
