// Tensor-core kernel family for chunkwise gated linear attention on sm_100a (Eq. attn_gla evaluated
// chunk by chunk, Section 3.5): tcgen05.mma (kind::tf32, fp32 accumulators in tensor memory) for
// every contraction, fp32 log-space cumulative gates.  bf16 storage, chunk = 64, d_k = d_v = 64.
//
// Why tf32 operands: the decayed operands q*exp(Lam), k*exp(-Lam), the masked scores and the
// chunk states are not bf16 numbers; rounding them to bf16 (8 significant bits) puts the maximum
// error at 2-3e-2 of the output RMS, above the 2e-2 parity bound, while tf32 (11 bits) stays below
// 1e-2 with the same fp32 accumulation.
//
// One CTA per (chunk, batch*head).  Operand tiles live in shared memory in the two swizzled
// formats of umma.cuh.  A 64 x 64 accumulator is produced as two 64 x 32 halves that share
// tensor-memory columns: the first half in lanes 0-15 of every 32-lane quarter, the second in
// lanes 16-31, so that every thread of a warp owns one accumulator row.
//
// Notation per chunk (rows j = 0..63 in scan order): Lam_j inclusive prefix sum of the gates,
// gamma = exp(Lam_63), Qt = q*exp(Lam), Kt = k*exp(-Lam), Kh = k*exp(Lam_63 - Lam),
// S = state entering the chunk, D = dL/d(state leaving the chunk), Dg = diag(gamma) D.
#include "dig_common.cuh"
#include "umma.cuh"

namespace dig {
namespace {

using namespace umma;
using bf16 = __nv_bfloat16;

constexpr int C = 64;          // chunk
constexpr int DK = 64, DV = 64;
constexpr int kTile = C * 64 * 4;        // bytes of one 64 x 64 operand tile
constexpr int kLamPitch = 68;            // floats; 16-byte aligned rows, conflict-free float4 reads

// Thread mappings for a CTA of 128*G threads; W = 32/G columns per thread.
//   load mapping : tile row `row`, columns [col0, col0 + W)
//   accumulator  : row `arow`, logical columns [acol0, acol0 + W), read from tensor-memory
//                  columns [acc + tcol, +W) of the warp's lane quarter
template <int G>
struct Ctx {
    static constexpr int W = 32 / G;
    int chunk, bh, b, h, tid, warp, lane;
    int row, seg, col0;
    int sub, arow, acol0, tcol;
};
template <int G>
__device__ __forceinline__ Ctx<G> make_ctx(const Geom &g)
{
    Ctx<G> c;
    c.chunk = blockIdx.x; c.bh = blockIdx.y; c.b = c.bh / g.H; c.h = c.bh - c.b * g.H;
    c.tid = threadIdx.x; c.warp = c.tid >> 5; c.lane = c.tid & 31;
    c.row = c.tid & 63; c.seg = c.tid >> 6; c.col0 = c.seg * Ctx<G>::W;
    c.sub = c.warp & 3;
    c.arow = 16 * c.sub + (c.lane & 15);
    c.tcol = Ctx<G>::W * (c.warp >> 2);
    c.acol0 = 32 * (c.lane >> 4) + c.tcol;
    return c;
}

// Token of tile row r, or -1 past the end of the sequence.
__device__ __forceinline__ int row_token(const Geom &g, int chunk, int r)
{
    const int p = chunk * C + r;
    return p < g.L ? scan_token(p, g.dir, g.gh, g.gw, g.L) : -1;
}

// W bf16 of one token row -> W floats (zeros for rows past the end).
template <int W>
__device__ __forceinline__ void load_row(const bf16 *base, const Geom &g, int b, int t, int h, int d, int col0,
                                         float (&f)[W])
{
    if (t < 0) {
#pragma unroll
        for (int i = 0; i < W; ++i) f[i] = 0.f;
        return;
    }
    const uint4 *p = reinterpret_cast<const uint4 *>(base + tok_offset(g, b, t, h, d) + col0);
#pragma unroll
    for (int j = 0; j < W / 8; ++j) {
        const uint4 u = __ldg(p + j);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[8 * j + 2 * i] = __uint_as_float(w[i] << 16);
            f[8 * j + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
}
template <int W>
__device__ __forceinline__ void load_row_f32(const float *p, float (&f)[W])
{
#pragma unroll
    for (int j = 0; j < W / 4; ++j) {
        const float4 u = __ldg(reinterpret_cast<const float4 *>(p) + j);
        f[4 * j] = u.x; f[4 * j + 1] = u.y; f[4 * j + 2] = u.z; f[4 * j + 3] = u.w;
    }
}

// Columns [col0, col0 + W) of `row`, rounded to tf32, into a K-format / M-format tile.
template <int W>
__device__ __forceinline__ void store_row_k(char *tile, int row, int col0, const float (&f)[W])
{
    char *base = tile + (col0 >> 5) * (C * 128) + row * 128;
    const int c16 = (col0 & 31) >> 2;
#pragma unroll
    for (int j = 0; j < W / 4; ++j)
        *reinterpret_cast<float4 *>(base + (((c16 + j) ^ (row & 7)) << 4)) =
            make_float4(to_tf32(f[4 * j]), to_tf32(f[4 * j + 1]), to_tf32(f[4 * j + 2]), to_tf32(f[4 * j + 3]));
}
template <int W>
__device__ __forceinline__ void store_row_m(char *tile, int row, int col0, const float (&f)[W])
{
    char *base = tile + (col0 >> 5) * (C * 128) + row * 128;
    const int c16 = (col0 & 31) >> 2;
#pragma unroll
    for (int j = 0; j < W / 4; ++j) {
        const int c = c16 + j;
        *reinterpret_cast<float4 *>(base + ((((c >> 1) ^ (row & 3)) << 5) | ((c & 1) << 4))) =
            make_float4(to_tf32(f[4 * j]), to_tf32(f[4 * j + 1]), to_tf32(f[4 * j + 2]), to_tf32(f[4 * j + 3]));
    }
}

// Gates of the chunk -> inclusive prefix sums in sLam[64][kLamPitch], Lam_63 in sLast[64].
// Thread (c = tid & 63, seg) owns W consecutive rows of channel c: W independent coalesced loads,
// a register prefix sum, one exchange of segment totals through sTot[2G][64].
template <int G>
__device__ __forceinline__ void chunk_gate_prefix(const float *__restrict__ gate, const Geom &g, const Ctx<G> &x,
                                                  float *sLam, float *sLast, float *sTot)
{
    constexpr int W = Ctx<G>::W, NSEG = 2 * G;
    const int c = x.row, seg = x.seg;
    float a[W];
#pragma unroll
    for (int j = 0; j < W; ++j) {
        const int t = row_token(g, x.chunk, W * seg + j);
        a[j] = t >= 0 ? __ldg(gate + tok_offset(g, x.b, t, x.h, DK) + c) : 0.f;
    }
#pragma unroll
    for (int j = 1; j < W; ++j) a[j] += a[j - 1];
    sTot[seg * 64 + c] = a[W - 1];
    __syncthreads();
    float add = 0.f;
#pragma unroll
    for (int s = 0; s < NSEG - 1; ++s)
        if (s < seg) add += sTot[s * 64 + c];
#pragma unroll
    for (int j = 0; j < W; ++j) sLam[(W * seg + j) * kLamPitch + c] = a[j] + add;
    if (seg == NSEG - 1) sLast[c] = a[W - 1] + add;
    __syncthreads();
}

template <int W>
__device__ __forceinline__ void read_lam(const float *sLam, int row, int col0, float (&lam)[W])
{
#pragma unroll
    for (int j = 0; j < W / 4; ++j) {
        const float4 v = *reinterpret_cast<const float4 *>(sLam + row * kLamPitch + col0 + 4 * j);
        lam[4 * j] = v.x; lam[4 * j + 1] = v.y; lam[4 * j + 2] = v.z; lam[4 * j + 3] = v.w;
    }
}

__device__ __forceinline__ char *align1024(char *p)
{
    return reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

struct Control {
    uint64_t bar[4];
    uint32_t tmem_base;
    uint32_t pad;
};

// Issues one 64 x 64 x 64 product as two 64 x 32 halves (see file header).  A_MN / B_MN: the
// operand tile is in M-format and read MN-major (contraction along its rows); otherwise it is in
// K-format and read K-major.
template <bool A_MN, bool B_MN>
__device__ __forceinline__ void issue_product(uint32_t d_tmem, uint32_t a_tile, uint32_t b_tile, bool accumulate)
{
    constexpr uint32_t idesc = idesc_tf32(64, 32, A_MN, B_MN);
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        const uint32_t d = d_tmem + ((uint32_t)(16 * hf) << 16);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
            const uint64_t da = A_MN ? desc_mnmajor<C>(a_tile, 8 * kk, 0) : desc_kmajor<C>(a_tile, 0, 8 * kk);
            const uint64_t db = B_MN ? desc_mnmajor<C>(b_tile, 8 * kk, 32 * hf) : desc_kmajor<C>(b_tile, 32 * hf, 8 * kk);
            mma_tf32(d, da, db, idesc, accumulate || kk > 0);
        }
    }
}

template <int G>
__device__ __forceinline__ void read_acc(uint32_t tmem_base, int acc_col, const Ctx<G> &x, float (&v)[Ctx<G>::W])
{
    tmem_ld(tmem_base + ((uint32_t)(32 * x.sub) << 16) + (uint32_t)(acc_col + x.tcol), v);
}

template <int W>
__device__ __forceinline__ void store_out(float *p, const float (&v)[W])
{
#pragma unroll
    for (int j = 0; j < W / 4; ++j)
        *reinterpret_cast<float4 *>(p + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}
template <int W>
__device__ __forceinline__ void store_out(bf16 *p, const float (&v)[W])
{
#pragma unroll
    for (int j = 0; j < W / 8; ++j) {
        uint4 u;
        __nv_bfloat162 t;
        t = __floats2bfloat162_rn(v[8 * j], v[8 * j + 1]); u.x = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]); u.y = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]); u.z = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]); u.w = *reinterpret_cast<uint32_t *>(&t);
        *reinterpret_cast<uint4 *>(p + 8 * j) = u;
    }
}

template <int G>
__device__ __forceinline__ void setup(Control *ctl, int nbar, uint32_t tmem_cols, const Ctx<G> &x)
{
    if (x.warp == 0) tmem_alloc(&ctl->tmem_base, tmem_cols);
    if (x.tid == 32) {
        for (int i = 0; i < nbar; ++i) mbar_init(&ctl->bar[i], 1);
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}
template <int G>
__device__ __forceinline__ void teardown(Control *ctl, uint32_t tmem_cols, const Ctx<G> &x)
{
    tc_fence_before_sync();
    __syncthreads();
    if (x.warp == 0) tmem_dealloc(ctl->tmem_base, tmem_cols);
}

// ---- kernel 1: chunk-local state contributions ----------------------------------------------
// U = Kh^T V (and W = Qt^T dO for the backward pass); gamma = exp(Lam_63).
template <int G, bool BWD>
__global__ void __launch_bounds__(128 * G)
tc_chunk_state(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
               const float *__restrict__ gate, const bf16 *__restrict__ d_out, float *__restrict__ states,
               float *__restrict__ gamma, float *__restrict__ dstates, int *status, Geom g)
{
    constexpr int W = Ctx<G>::W;
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    constexpr int nTiles = BWD ? 4 : 2;
    char *tKh = base, *tV = base + kTile, *tQ = base + 2 * kTile, *tG = base + 3 * kTile;    // all M-format
    float *sLam = reinterpret_cast<float *>(base + nTiles * kTile);
    float *sLast = sLam + C * kLamPitch, *sTot = sLast + 64;
    Control *ctl = reinterpret_cast<Control *>(sTot + 2 * G * 64);
    const Ctx<G> x = make_ctx<G>(g);
    constexpr uint32_t kCols = BWD ? 64 : 32;
    setup(ctl, 1, kCols, x);

    const int t = row_token(g, x.chunk, x.row);
    float kk[W], vv[W], qq[W], gg[W];
    load_row<W>(k, g, x.b, t, x.h, DK, x.col0, kk);
    load_row<W>(v, g, x.b, t, x.h, DV, x.col0, vv);
    if (BWD) {
        load_row<W>(q, g, x.b, t, x.h, DK, x.col0, qq);
        load_row<W>(d_out, g, x.b, t, x.h, DV, x.col0, gg);
    }
    chunk_gate_prefix<G>(gate, g, x, sLam, sLast, sTot);
    const size_t chunk_id = (size_t)x.bh * g.N + x.chunk;
    if (x.tid < 64) gamma[chunk_id * DK + x.tid] = __expf(sLast[x.tid]);
    {
        float lam[W];
        read_lam<W>(sLam, x.row, x.col0, lam);
#pragma unroll
        for (int i = 0; i < W; ++i) {
            if (BWD) qq[i] *= __expf(lam[i]);
            kk[i] *= __expf(sLast[x.col0 + i] - lam[i]);
        }
        store_row_m<W>(tKh, x.row, x.col0, kk);
        store_row_m<W>(tV, x.row, x.col0, vv);
        if (BWD) {
            store_row_m<W>(tQ, x.row, x.col0, qq);
            store_row_m<W>(tG, x.row, x.col0, gg);
        }
    }
    fence_async_smem();
    __syncthreads();
    const uint32_t tmem = ctl->tmem_base;
    if (x.tid == 0) {
        tc_fence_after_sync();
        issue_product<true, true>(tmem, smem_u32(tKh), smem_u32(tV), false);
        if (BWD) issue_product<true, true>(tmem + 32, smem_u32(tQ), smem_u32(tG), false);
        mma_commit(&ctl->bar[0]);
    }
    if (mbar_wait(&ctl->bar[0], 0, status)) {
        tc_fence_after_sync();
        float acc[W];
        read_acc<G>(tmem, 0, x, acc);
        store_out<W>(states + chunk_id * DK * DV + x.arow * DV + x.acol0, acc);
        if (BWD) {
            read_acc<G>(tmem, 32, x, acc);
            store_out<W>(dstates + chunk_id * DK * DV + x.arow * DV + x.acol0, acc);
        }
    }
    teardown(ctl, kCols, x);
}

// ---- kernel 3: outputs ---------------------------------------------------------------------------
// out = tril(Qt Kt^T) V + Qt S
template <int G, typename TO>
__global__ void __launch_bounds__(128 * G)
tc_chunk_out(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
             const float *__restrict__ gate, const float *__restrict__ states, TO *__restrict__ out,
             int *status, Geom g)
{
    constexpr int W = Ctx<G>::W;
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    char *tQ = base, *tK = base + kTile, *tP = base + 2 * kTile;      // K-format
    char *tV = base + 3 * kTile, *tS = base + 4 * kTile;             // M-format
    float *sLam = reinterpret_cast<float *>(base + 5 * kTile);
    float *sLast = sLam + C * kLamPitch, *sTot = sLast + 64;
    Control *ctl = reinterpret_cast<Control *>(sTot + 2 * G * 64);
    const Ctx<G> x = make_ctx<G>(g);
    constexpr uint32_t kCols = 64;
    setup(ctl, 2, kCols, x);

    const int t = row_token(g, x.chunk, x.row);
    const size_t chunk_id = (size_t)x.bh * g.N + x.chunk;
    float qq[W], kk[W], vv[W], ss[W];
    load_row<W>(q, g, x.b, t, x.h, DK, x.col0, qq);
    load_row<W>(k, g, x.b, t, x.h, DK, x.col0, kk);
    load_row<W>(v, g, x.b, t, x.h, DV, x.col0, vv);
    load_row_f32<W>(states + chunk_id * DK * DV + x.row * DV + x.col0, ss);
    chunk_gate_prefix<G>(gate, g, x, sLam, sLast, sTot);
    {
        float lam[W];
        read_lam<W>(sLam, x.row, x.col0, lam);
#pragma unroll
        for (int i = 0; i < W; ++i) {
            qq[i] *= __expf(lam[i]);
            kk[i] *= __expf(-lam[i]);
        }
        store_row_k<W>(tQ, x.row, x.col0, qq);
        store_row_k<W>(tK, x.row, x.col0, kk);
    }
    fence_async_smem();
    __syncthreads();
    const uint32_t tmem = ctl->tmem_base;
    if (x.tid == 0) {
        tc_fence_after_sync();
        issue_product<false, false>(tmem, smem_u32(tQ), smem_u32(tK), false);      // scores
        mma_commit(&ctl->bar[0]);
    }
    store_row_m<W>(tV, x.row, x.col0, vv);       // staged while the scores are computed
    store_row_m<W>(tS, x.row, x.col0, ss);
    const bool ok = mbar_wait(&ctl->bar[0], 0, status);
    if (ok) {
        tc_fence_after_sync();
        float p[W];
        read_acc<G>(tmem, 0, x, p);
#pragma unroll
        for (int j = 0; j < W; ++j)
            if (x.acol0 + j > x.arow) p[j] = 0.f;            // keep s <= t; the diagonal has weight 1
        store_row_k<W>(tP, x.arow, x.acol0, p);
    }
    fence_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (x.tid == 0 && ok) {
        tc_fence_after_sync();
        issue_product<false, true>(tmem + 32, smem_u32(tP), smem_u32(tV), false);
        issue_product<false, true>(tmem + 32, smem_u32(tQ), smem_u32(tS), true);
        mma_commit(&ctl->bar[1]);
    }
    if (ok && mbar_wait(&ctl->bar[1], 0, status)) {
        tc_fence_after_sync();
        float o[W];
        read_acc<G>(tmem, 32, x, o);
        const int to = row_token(g, x.chunk, x.arow);
        if (to >= 0) store_out<W>(out + tok_offset(g, x.b, to, x.h, DV) + x.acol0, o);
    }
    teardown(ctl, kCols, x);
}

// ---- kernel 4: gradients ---------------------------------------------------------------------------
//   P  = tril(Qt Kt^T),  dP = tril(dO V^T)
//   dq = (dP Kt + dO S^T) * exp(Lam)
//   dk = (dP^T Qt + V Dg^T) * exp(-Lam)
//   dv = P^T dO + Kt Dg
//   dgate_j = carry + sum_{r >= j in chunk} (q*dq - k*dk)_r
template <int G, typename TO>
__global__ void __launch_bounds__(128 * G)
tc_chunk_bwd(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
             const float *__restrict__ gate, const bf16 *__restrict__ d_out, const float *__restrict__ states,
             const float *__restrict__ dstates, const float *__restrict__ carry, TO *__restrict__ dq,
             TO *__restrict__ dk, TO *__restrict__ dv, float *__restrict__ dgate, int *status, Geom g)
{
    constexpr int W = Ctx<G>::W;
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    // K-format tiles
    char *tQk = base + 0 * kTile, *tKk = base + 1 * kTile, *tVk = base + 2 * kTile, *tGk = base + 3 * kTile;
    char *tSk = base + 4 * kTile, *tDk = base + 5 * kTile, *tdPk = base + 6 * kTile;
    // M-format tiles
    char *tQm = base + 7 * kTile, *tKm = base + 8 * kTile, *tGm = base + 9 * kTile, *tDm = base + 10 * kTile;
    char *tdPm = base + 11 * kTile;
    char *tPm = tQk;                          // scores overwrite Qt (K-format) once P = Qt Kt^T is done
    float *sX = reinterpret_cast<float *>(tSk);   // q*dq - k*dk, after every product has completed
    float *sLam = reinterpret_cast<float *>(base + 12 * kTile);
    float *sLast = sLam + C * kLamPitch, *sTot = sLast + 64;
    Control *ctl = reinterpret_cast<Control *>(sTot + 2 * G * 64);
    const Ctx<G> x = make_ctx<G>(g);
    constexpr uint32_t kCols = 256;
    constexpr int aP = 0, adP = 32, adQ = 64, adK = 96, adV = 128;      // accumulator columns
    setup(ctl, 2, kCols, x);

    const int t = row_token(g, x.chunk, x.row);
    const size_t chunk_id = (size_t)x.bh * g.N + x.chunk;
    {
        float qq[W], kk[W], vv[W], gg[W], ss[W], dd[W];
        load_row<W>(q, g, x.b, t, x.h, DK, x.col0, qq);
        load_row<W>(k, g, x.b, t, x.h, DK, x.col0, kk);
        load_row<W>(v, g, x.b, t, x.h, DV, x.col0, vv);
        load_row<W>(d_out, g, x.b, t, x.h, DV, x.col0, gg);
        load_row_f32<W>(states + chunk_id * DK * DV + x.row * DV + x.col0, ss);
        load_row_f32<W>(dstates + chunk_id * DK * DV + x.row * DV + x.col0, dd);
        chunk_gate_prefix<G>(gate, g, x, sLam, sLast, sTot);
        float lam[W];
        read_lam<W>(sLam, x.row, x.col0, lam);
        const float gm = __expf(sLast[x.row]);           // state tiles are indexed [key channel][value channel]
#pragma unroll
        for (int i = 0; i < W; ++i) {
            qq[i] *= __expf(lam[i]);
            kk[i] *= __expf(-lam[i]);
            dd[i] *= gm;
        }
        store_row_k<W>(tQk, x.row, x.col0, qq);
        store_row_m<W>(tQm, x.row, x.col0, qq);
        store_row_k<W>(tKk, x.row, x.col0, kk);
        store_row_m<W>(tKm, x.row, x.col0, kk);
        store_row_k<W>(tVk, x.row, x.col0, vv);
        store_row_k<W>(tGk, x.row, x.col0, gg);
        store_row_m<W>(tGm, x.row, x.col0, gg);
        store_row_k<W>(tSk, x.row, x.col0, ss);
        store_row_k<W>(tDk, x.row, x.col0, dd);
        store_row_m<W>(tDm, x.row, x.col0, dd);
    }
    fence_async_smem();
    __syncthreads();
    const uint32_t tmem = ctl->tmem_base;
    if (x.tid == 0) {
        tc_fence_after_sync();
        issue_product<false, false>(tmem + aP, smem_u32(tQk), smem_u32(tKk), false);     // P  = Qt Kt^T
        issue_product<false, false>(tmem + adP, smem_u32(tGk), smem_u32(tVk), false);    // dP = dO V^T
        mma_commit(&ctl->bar[0]);
        issue_product<false, false>(tmem + adQ, smem_u32(tGk), smem_u32(tSk), false);    // dO S^T
        issue_product<false, false>(tmem + adK, smem_u32(tVk), smem_u32(tDk), false);    // V Dg^T
        issue_product<false, true>(tmem + adV, smem_u32(tKk), smem_u32(tDm), false);     // Kt Dg
    }
    const bool ok = mbar_wait(&ctl->bar[0], 0, status);
    if (ok) {
        tc_fence_after_sync();
        float p[W];
        read_acc<G>(tmem, aP, x, p);
#pragma unroll
        for (int j = 0; j < W; ++j)
            if (x.acol0 + j > x.arow) p[j] = 0.f;
        store_row_m<W>(tPm, x.arow, x.acol0, p);
        read_acc<G>(tmem, adP, x, p);
#pragma unroll
        for (int j = 0; j < W; ++j)
            if (x.acol0 + j > x.arow) p[j] = 0.f;
        store_row_k<W>(tdPk, x.arow, x.acol0, p);
        store_row_m<W>(tdPm, x.arow, x.acol0, p);
    }
    fence_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (x.tid == 0 && ok) {
        tc_fence_after_sync();
        issue_product<false, true>(tmem + adQ, smem_u32(tdPk), smem_u32(tKm), true);     // + dP Kt
        issue_product<true, true>(tmem + adK, smem_u32(tdPm), smem_u32(tQm), true);      // + dP^T Qt
        issue_product<true, true>(tmem + adV, smem_u32(tPm), smem_u32(tGm), true);       // + P^T dO
        mma_commit(&ctl->bar[1]);
    }
    const bool ok2 = ok && mbar_wait(&ctl->bar[1], 0, status);
    if (ok2) {
        tc_fence_after_sync();
        const int to = row_token(g, x.chunk, x.arow);
        float a[W], lam[W], xq[W];
        read_lam<W>(sLam, x.arow, x.acol0, lam);
        read_acc<G>(tmem, adQ, x, a);
#pragma unroll
        for (int i = 0; i < W; ++i) a[i] *= __expf(lam[i]);
        if (to >= 0) {
            store_out<W>(dq + tok_offset(g, x.b, to, x.h, DK) + x.acol0, a);
            float r[W];
            load_row<W>(q, g, x.b, to, x.h, DK, x.acol0, r);
#pragma unroll
            for (int i = 0; i < W; ++i) xq[i] = r[i] * a[i];
        } else {
#pragma unroll
            for (int i = 0; i < W; ++i) xq[i] = 0.f;
        }
        read_acc<G>(tmem, adK, x, a);
#pragma unroll
        for (int i = 0; i < W; ++i) a[i] *= __expf(-lam[i]);
        if (to >= 0) {
            store_out<W>(dk + tok_offset(g, x.b, to, x.h, DK) + x.acol0, a);
            float r[W];
            load_row<W>(k, g, x.b, to, x.h, DK, x.acol0, r);
#pragma unroll
            for (int i = 0; i < W; ++i) xq[i] -= r[i] * a[i];
        }
#pragma unroll
        for (int j = 0; j < W / 4; ++j)
            *reinterpret_cast<float4 *>(sX + x.arow * kLamPitch + x.acol0 + 4 * j) =
                make_float4(xq[4 * j], xq[4 * j + 1], xq[4 * j + 2], xq[4 * j + 3]);
        read_acc<G>(tmem, adV, x, a);
        if (to >= 0) store_out<W>(dv + tok_offset(g, x.b, to, x.h, DV) + x.acol0, a);
    }
    if (__syncthreads_and(ok2)) {      // uniform: either every thread saw both products finish or none continues
        // gate gradient: suffix sums of x down the chunk (W rows per thread, segment totals exchanged
        // through shared memory) plus what later chunks carry in
        const int c = x.row, seg = x.seg;
        float s[W];
#pragma unroll
        for (int j = 0; j < W; ++j) s[j] = sX[(W * seg + j) * kLamPitch + c];
#pragma unroll
        for (int j = W - 2; j >= 0; --j) s[j] += s[j + 1];
        sTot[seg * 64 + c] = s[0];
        __syncthreads();
        float add = __ldg(carry + chunk_id * DK + c);
#pragma unroll
        for (int sg = 1; sg < 2 * G; ++sg)
            if (sg > seg) add += sTot[sg * 64 + c];
#pragma unroll
        for (int j = 0; j < W; ++j) {
            const int tj = row_token(g, x.chunk, W * seg + j);
            if (tj >= 0) dgate[tok_offset(g, x.b, tj, x.h, DK) + c] = s[j] + add;
        }
    }
    teardown(ctl, kCols, x);
}

template <int G>
constexpr size_t smem_bytes(int tiles)
{
    return 1024 + (size_t)tiles * kTile + sizeof(float) * (C * kLamPitch + 64 + 2 * G * 64) + sizeof(Control);
}

template <typename K>
dig_status opt_in(K kernel, size_t bytes)
{
    return cuda_ok(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
}

constexpr int GF = 1;      // thread groups of the forward kernels (128 threads, two CTAs per SM)
constexpr int GB = 2;      // backward kernel: 256 threads, one CTA per SM

template <typename TO>
dig_status fwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, false);
    int *status = device_status_ptr();
    if (!status) return DIG_ERR_CUDA;
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = tc_chunk_state<GF, false>;
    auto k3 = tc_chunk_out<GF, TO>;
    if ((st = opt_in(k1, smem_bytes<GF>(2))) != DIG_OK) return st;
    if ((st = opt_in(k3, smem_bytes<GF>(5))) != DIG_OK) return st;
    {
        KernelTimer t(KID_TC_STATE, a.stream);
        k1<<<grid, 128 * GF, smem_bytes<GF>(2), a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v,
                                                            a.gate, nullptr, w.states, w.gamma, nullptr, status, g);
    }
    if ((st = launch_state_scan_fwd(w, g, a.stream)) != DIG_OK) return st;
    KernelTimer t(KID_TC_OUT, a.stream);
    k3<<<grid, 128 * GF, smem_bytes<GF>(5), a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate,
                                                        w.states, (TO *)a.out, status, g);
    return cuda_ok(cudaGetLastError());
}

template <typename TO>
dig_status bwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, true);
    int *status = device_status_ptr();
    if (!status) return DIG_ERR_CUDA;
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = tc_chunk_state<GF, true>;
    auto k4 = tc_chunk_bwd<GB, TO>;
    if ((st = opt_in(k1, smem_bytes<GF>(4))) != DIG_OK) return st;
    if ((st = opt_in(k4, smem_bytes<GB>(12))) != DIG_OK) return st;
    {
        KernelTimer t(KID_TC_STATE, a.stream);
        k1<<<grid, 128 * GF, smem_bytes<GF>(4), a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v,
                                                            a.gate, (const bf16 *)a.d_out, w.states, w.gamma, w.dstates,
                                                            status, g);
    }
    if ((st = launch_state_scan_fwd(w, g, a.stream)) != DIG_OK) return st;
    if ((st = launch_state_scan_bwd(w, g, a.stream)) != DIG_OK) return st;
    KernelTimer t(KID_TC_BWD, a.stream);
    k4<<<grid, 128 * GB, smem_bytes<GB>(12), a.stream>>>(
        (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate, (const bf16 *)a.d_out, w.states, w.dstates,
        w.carry, (TO *)a.dq, (TO *)a.dk, (TO *)a.dv, a.dgate, status, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

bool tensor_supports(int dk, int dv, int chunk, int dtype, bool backward)
{
    (void)backward;
    if (dtype != DIG_BF16 && dtype != DIG_BF16_F32OUT) return false;
    return dk == DK && dv == DV && chunk == C;
}

dig_status tensor_gla_fwd(const GlaArgs &a)
{
    return a.dtype == DIG_BF16 ? fwd_typed<bf16>(a) : fwd_typed<float>(a);
}

dig_status tensor_gla_bwd(const GlaArgs &a)
{
    return a.dtype == DIG_BF16 ? bwd_typed<bf16>(a) : bwd_typed<float>(a);
}

}  // namespace dig
