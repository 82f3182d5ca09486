// Output gate of the GLA layer (Eq. attn_gla, the line that forms Y_t before the projection W_O):
//     z = Swish(r) (.) LN(o)      per (token, head) row of d_v values,
// and its reverse mode.  Elementwise plus two row reductions, so bandwidth-bound: a row is held by 8
// (d_v <= 64), 9 (d_v = 72: three rows per warp, five lanes idle) or 16 lanes of a warp with 8
// consecutive values each (16-byte loads of bf16, 2 x 16 of fp32), the row statistics come from
// shuffles inside that lane group, every tensor is read once and written once.  The affine gradients are summed per CTA in registers and shared memory and then
// across CTAs by a second kernel in a fixed order.
#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int kThreads = 256;
// Grid caps (measured): the reverse kernel does best with as many CTAs as stay resident together, three
// per SM at its register count, so that the grid-stride loops end together and not in a ragged last
// wave; the forward kernel does best with eight per SM.
constexpr int kFwdPerSM = 8, kBwdPerSM = 3;

__device__ __forceinline__ void load8(const float *p, float (&f)[8])
{
    const float4 a = load4(p), b = load4(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&f)[8])
{
    const uint4 u = *reinterpret_cast<const uint4 *>(p);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
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

// Thread -> (row slot of the CTA, lane of the row's group): 32 / LPR rows per warp.
template <int LPR>
struct RowMap {
    static constexpr int kRowsPerWarp = 32 / LPR, kRows = (kThreads / 32) * kRowsPerWarp;
    int lane, slot, gbase;      // lane in the group, row slot, first warp lane of the group
    bool valid;                 // false for the warp's left-over lanes when LPR is not a power of two
    __device__ __forceinline__ RowMap()
    {
        const int l = threadIdx.x & 31, grp = l / LPR;
        lane = l - grp * LPR;
        gbase = grp * LPR;
        valid = grp < kRowsPerWarp;
        slot = (threadIdx.x >> 5) * kRowsPerWarp + (valid ? grp : 0);
    }
};
// Sum over the row's lane group, returned to all of its lanes.  Power-of-two groups: butterfly.  Nine
// lanes: the ninth is folded into the first, a butterfly over the first eight, then a broadcast.
template <int LPR> __device__ __forceinline__ float group_sum(float x, const RowMap<LPR> &m)
{
    if ((LPR & (LPR - 1)) == 0) {
#pragma unroll
        for (int k = LPR / 2; k >= 1; k >>= 1) x += __shfl_xor_sync(0xffffffffu, x, k);
        return x;
    }
    static_assert((LPR & (LPR - 1)) == 0 || LPR == 9, "lane groups of a power of two or of nine");
    const float y = __shfl_sync(0xffffffffu, x, min(m.gbase + 8, 31));
    if (m.lane == 0) x += y;
#pragma unroll
    for (int k = 4; k >= 1; k >>= 1) {
        const float t = __shfl_sync(0xffffffffu, x, min(m.gbase + ((m.lane ^ k) & 7), 31));
        if (m.lane < 8) x += t;
    }
    return __shfl_sync(0xffffffffu, x, m.gbase);
}

// Normalised row n = (o - mean) * rstd of the lane's 8 columns (zero where the lane holds none).
template <int LPR> __device__ __forceinline__ float normalise(const float (&o)[8], bool has, float inv_d, float eps,
                                                               float (&n)[8], const RowMap<LPR> &m)
{
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) s += o[e];
    const float mean = group_sum<LPR>(s, m) * inv_d;
    float v = 0.f;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        n[e] = has ? o[e] - mean : 0.f;
        v = fmaf(n[e], n[e], v);
    }
    const float rstd = rsqrtf(group_sum<LPR>(v, m) * inv_d + eps);
#pragma unroll
    for (int e = 0; e < 8; ++e) n[e] *= rstd;
    return rstd;
}

// 1 / (1 + e^-r) with the fast exponential and the fast reciprocal (2 ulp each; e^-r = inf gives 0)
__device__ __forceinline__ float sigmoidf(float r) { return __fdividef(1.f, 1.f + __expf(-r)); }

// TA: type of o (the GLA output: input storage type when it comes from memory written by a caller, output
// storage type when it comes straight from the forward pass), TR: type of r, TZ: type of z.  o and z may
// be the same buffer: a lane reads its values of a row before it writes them.
template <typename TA, typename TR, typename TZ, int LPR>
__global__ void __launch_bounds__(kThreads)
outgate_fwd(const TA *o, const TR *__restrict__ r, const float *__restrict__ ln_w,
            const float *__restrict__ ln_b, TZ *z, long long rows, int dv, float eps)
{
    constexpr int kRows = RowMap<LPR>::kRows;
    const RowMap<LPR> rm;
    const int slot = rm.slot, col = rm.lane * 8;
    const bool has_col = rm.valid && col < dv;
    const float inv_d = 1.f / (float)dv;
    float w[8], b[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        w[e] = (ln_w != nullptr && has_col) ? ln_w[col + e] : 1.f;
        b[e] = (ln_b != nullptr && has_col) ? ln_b[col + e] : 0.f;
    }
    pdl_wait();
    pdl_launch_dependents();
    for (long long base = (long long)blockIdx.x * kRows; base < rows; base += (long long)gridDim.x * kRows) {
        const long long row = base + slot;
        const bool has = has_col && row < rows;
        float ov[8] = {0, 0, 0, 0, 0, 0, 0, 0}, rv[8] = {0, 0, 0, 0, 0, 0, 0, 0}, n[8];
        if (has) {
            load8(o + row * dv + col, ov);
            load8(r + row * dv + col, rv);
        }
        normalise<LPR>(ov, has, inv_d, eps, n, rm);
        float out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = rv[e] * sigmoidf(rv[e]) * fmaf(n[e], w[e], b[e]);
        if (has) store8(z + row * dv + col, out);
    }
}

template <typename TI, typename TO, int LPR>
__global__ void __launch_bounds__(kThreads)
outgate_bwd(const TI *__restrict__ o, const TI *__restrict__ r, const TI *__restrict__ dz,
            const float *__restrict__ ln_w, const float *__restrict__ ln_b, TO *__restrict__ d_o,
            TO *__restrict__ d_r, float *__restrict__ partial, long long rows, int dv, float eps)
{
    constexpr int kRows = RowMap<LPR>::kRows;
    __shared__ float red[kRows][2][LPR * 8];
    const RowMap<LPR> rm;
    const int slot = rm.slot, col = rm.lane * 8;
    const bool has_col = rm.valid && col < dv;
    const float inv_d = 1.f / (float)dv;
    float w[8], b[8], aw[8], ab[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        w[e] = (ln_w != nullptr && has_col) ? ln_w[col + e] : 1.f;
        b[e] = (ln_b != nullptr && has_col) ? ln_b[col + e] : 0.f;
        aw[e] = ab[e] = 0.f;
    }
    pdl_wait();
    pdl_launch_dependents();
    for (long long base = (long long)blockIdx.x * kRows; base < rows; base += (long long)gridDim.x * kRows) {
        const long long row = base + slot;
        const bool has = has_col && row < rows;
        float ov[8] = {0, 0, 0, 0, 0, 0, 0, 0}, rv[8] = {0, 0, 0, 0, 0, 0, 0, 0}, gv[8] = {0, 0, 0, 0, 0, 0, 0, 0}, n[8];
        if (has) {
            load8(o + row * dv + col, ov);
            load8(r + row * dv + col, rv);
            load8(dz + row * dv + col, gv);
        }
        const float rstd = normalise<LPR>(ov, has, inv_d, eps, n, rm);
        float dr[8], dn[8], s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float sg = sigmoidf(rv[e]);
            const float y = fmaf(n[e], w[e], b[e]);
            dr[e] = gv[e] * y * fmaf(rv[e] * sg, 1.f - sg, sg);
            const float dy = gv[e] * rv[e] * sg;                 // zero where the lane holds no value
            aw[e] = fmaf(dy, n[e], aw[e]);
            ab[e] += dy;
            dn[e] = dy * w[e];
            s1 += dn[e];
            s2 = fmaf(dn[e], n[e], s2);
        }
        const float m1 = group_sum<LPR>(s1, rm) * inv_d, m2 = group_sum<LPR>(s2, rm) * inv_d;
        float dov[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) dov[e] = rstd * (dn[e] - m1 - n[e] * m2);
        if (has) {
            store8(d_o + row * dv + col, dov);
            store8(d_r + row * dv + col, dr);
        }
    }
    if (partial == nullptr) return;
    if (rm.valid) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            red[slot][0][col + e] = aw[e];
            red[slot][1][col + e] = ab[e];
        }
    }
    __syncthreads();
    // partial[cta][2][dv]
    for (int idx = threadIdx.x; idx < 2 * LPR * 8; idx += kThreads) {
        const int which = idx / (LPR * 8), c = idx - which * (LPR * 8);
        if (c >= dv) continue;
        float sum = 0.f;
#pragma unroll 8
        for (int s = 0; s < kRows; ++s) sum += red[s][which][c];
        partial[((size_t)blockIdx.x * 2 + which) * dv + c] = sum;
    }
}

// One warp per parameter: its lanes add every 32nd partial sum, then a butterfly (a fixed order, so the
// result does not depend on scheduling).
__global__ void __launch_bounds__(256)
outgate_affine_sum(const float *__restrict__ partial, float *__restrict__ dln_w, float *__restrict__ dln_b,
                   int nctas, int dv)
{
    pdl_wait();
    pdl_launch_dependents();
    const int idx = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (idx >= 2 * dv) return;          // uniform over the warp
    float sum = 0.f;
    for (int s = lane; s < nctas; s += 32) sum += partial[(size_t)s * 2 * dv + idx];
#pragma unroll
    for (int k = 16; k >= 1; k >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, k);
    if (lane != 0) return;
    if (idx < dv) {
        if (dln_w != nullptr) dln_w[idx] = sum;
    } else if (dln_b != nullptr) {
        dln_b[idx - dv] = sum;
    }
}

// lanes per row for a row length
int lanes_for(int dv) { return dv <= 64 ? 8 : dv == 72 ? 9 : 16; }
int grid_for(long long rows, int lpr, int per_sm = kBwdPerSM)
{
    int sms = device_sm_count();
    if (sms <= 0) sms = 148;            // sizing call without a device: the count the launch will most likely see
    const int kMaxCtas = sms * per_sm;
    const long long per = (kThreads / 32) * (32 / lpr), need = (rows + per - 1) / per;
    return (int)(need < kMaxCtas ? need : kMaxCtas);
}

template <typename TA, typename TR, typename TZ>
void fwd_dispatch3(const void *o, const void *r, const float *w, const float *b, void *z, long long rows, int dv,
                   float eps, cudaStream_t stream)
{
    if (dv <= 64)
        launch_pdl(outgate_fwd<TA, TR, TZ, 8>, dim3(grid_for(rows, 8, kFwdPerSM)), dim3(kThreads), 0, stream, (const TA *)o,
                   (const TR *)r, w, b, (TZ *)z, rows, dv, eps);
    else if (dv == 72)
        launch_pdl(outgate_fwd<TA, TR, TZ, 9>, dim3(grid_for(rows, 9, kFwdPerSM)), dim3(kThreads), 0, stream, (const TA *)o,
                   (const TR *)r, w, b, (TZ *)z, rows, dv, eps);
    else
        launch_pdl(outgate_fwd<TA, TR, TZ, 16>, dim3(grid_for(rows, 16, kFwdPerSM)), dim3(kThreads), 0, stream, (const TA *)o,
                   (const TR *)r, w, b, (TZ *)z, rows, dv, eps);
}
template <typename TI, typename TO>
void fwd_dispatch(const void *o, const void *r, const float *w, const float *b, void *z, long long rows, int dv,
                  float eps, cudaStream_t stream)
{
    fwd_dispatch3<TI, TI, TO>(o, r, w, b, z, rows, dv, eps, stream);
}

template <typename TI, typename TO>
void bwd_dispatch(const void *o, const void *r, const void *dz, const float *w, const float *b, void *d_o, void *d_r,
                  float *partial, long long rows, int dv, float eps, cudaStream_t stream)
{
    if (dv <= 64)
        launch_pdl(outgate_bwd<TI, TO, 8>, dim3(grid_for(rows, 8)), dim3(kThreads), 0, stream, (const TI *)o,
                   (const TI *)r, (const TI *)dz, w, b, (TO *)d_o, (TO *)d_r, partial, rows, dv, eps);
    else if (dv == 72)
        launch_pdl(outgate_bwd<TI, TO, 9>, dim3(grid_for(rows, 9)), dim3(kThreads), 0, stream, (const TI *)o,
                   (const TI *)r, (const TI *)dz, w, b, (TO *)d_o, (TO *)d_r, partial, rows, dv, eps);
    else
        launch_pdl(outgate_bwd<TI, TO, 16>, dim3(grid_for(rows, 16)), dim3(kThreads), 0, stream, (const TI *)o,
                   (const TI *)r, (const TI *)dz, w, b, (TO *)d_o, (TO *)d_r, partial, rows, dv, eps);
}

}  // namespace

size_t outgate_bwd_workspace_bytes(long long rows, int dv)
{
    return (size_t)grid_for(rows, lanes_for(dv)) * 2 * (size_t)dv * sizeof(float);
}

dig_status launch_outgate_fwd(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                              long long rows, int dv, float eps, int dtype, cudaStream_t stream)
{
    KernelTimer t(KID_OUTGATE, stream);
    if (dtype == DIG_F32) fwd_dispatch<float, float>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    else if (dtype == DIG_BF16) fwd_dispatch<__nv_bfloat16, __nv_bfloat16>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    else fwd_dispatch<__nv_bfloat16, float>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    return cuda_ok(cudaGetLastError());
}

// o in the output storage type of `dtype` (as the forward pass writes it), r in the input storage type.
dig_status launch_outgate_fwd_mixed(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                                    long long rows, int dv, float eps, int dtype, cudaStream_t stream)
{
    KernelTimer t(KID_OUTGATE, stream);
    if (dtype == DIG_F32) fwd_dispatch3<float, float, float>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    else if (dtype == DIG_BF16) fwd_dispatch3<__nv_bfloat16, __nv_bfloat16, __nv_bfloat16>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    else fwd_dispatch3<float, __nv_bfloat16, float>(o, r, ln_w, ln_b, z, rows, dv, eps, stream);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_outgate_bwd(const void *o, const void *r, const void *dz, const float *ln_w, const float *ln_b,
                              void *d_o, void *d_r, float *dln_w, float *dln_b, long long rows, int dv, float eps,
                              int dtype, float *partial, cudaStream_t stream)
{
    const bool affine = dln_w != nullptr || dln_b != nullptr;
    float *part = affine ? partial : nullptr;
    {
        KernelTimer t(KID_OUTGATE, stream);
        if (dtype == DIG_F32) bwd_dispatch<float, float>(o, r, dz, ln_w, ln_b, d_o, d_r, part, rows, dv, eps, stream);
        else if (dtype == DIG_BF16)
            bwd_dispatch<__nv_bfloat16, __nv_bfloat16>(o, r, dz, ln_w, ln_b, d_o, d_r, part, rows, dv, eps, stream);
        else bwd_dispatch<__nv_bfloat16, float>(o, r, dz, ln_w, ln_b, d_o, d_r, part, rows, dv, eps, stream);
    }
    if (cudaGetLastError() != cudaSuccess) return DIG_ERR_CUDA;
    if (!affine) return DIG_OK;
    KernelTimer t(KID_OUTGATE, stream);
    launch_pdl(outgate_affine_sum, dim3((2 * dv + 7) / 8), dim3(256), 0, stream, (const float *)partial, dln_w,
               dln_b, grid_for(rows, lanes_for(dv)), dv);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
