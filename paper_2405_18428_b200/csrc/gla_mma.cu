// Warp-MMA kernel family for chunkwise gated linear attention (Eq. attn_gla, evaluated chunk by chunk
// as Section 3.5 describes): serves bf16 requests whose head size or chunk size the tcgen05 family
// does not cover (any d_k, d_v that is a multiple of 8 up to 128, chunks of 16, 32, 64 or 128 tokens
// as far as shared memory allows), e.g. the 72-wide heads of the largest model.  Same decomposition
// as the other families: per-chunk state contributions, a scan over the chunks, then one CTA per
// (chunk, batch*head) for the outputs or the gradients.  Every contraction runs on the tensor cores
// through mma.sync.m16n8k8 (tf32 operands, fp32 accumulation) with fragments read straight from
// padded fp32 tiles in shared memory, so any multiple of 8 works as a contraction length and any
// multiple of 16 (after zero padding) as an output extent.  Operands are rounded to tf32 when the
// tiles are filled.  Requests in fp32 storage (served here only with the value-channel gate) keep full
// fp32 tiles instead and split every operand at fragment load into a tf32 head and a tf32 tail,
// x = hi + lo: three products hi*hi + lo*hi + hi*lo per fragment pair leave errors of order 2^-21,
// the accuracy fp32 storage is held to.
//
// Notation per chunk (rows j = 0..C-1 in scan order, zero rows past the end of the sequence):
//   Lam_j = inclusive prefix sum of the gates, gamma = exp(Lam_{C-1}),
//   Qt = q*exp(Lam), Kt = k*exp(-Lam), Kh = k*exp(Lam_{C-1}-Lam),
//   S = state entering the chunk, Dg = diag(gamma) * dL/d(state leaving the chunk); the scan kernels
//   leave both rounded to tf32 in the workspace.
#include <type_traits>

#include "dig_common.cuh"

namespace dig {
namespace {

using bf16 = __nv_bfloat16;
constexpr int kThreads = 512, kWarps = kThreads / 32;
constexpr int kMaxNB = 8;                    // 8-column fragments per warp tile: up to 64 columns

__host__ __device__ constexpr int pad16(int d) { return (d + 15) & ~15; }
// Row pitch (floats) of a tile whose rows hold `d` values: a multiple of 4 whose quarter is odd, so the
// 8 rows x 4 columns a fragment load touches fall into 32 different banks.
__host__ __device__ constexpr int pitch(int d) { return pad16(d) + 4; }
// The same for tiles whose padding columns are never read (every kernel but the state kernel, where d_k
// is an output extent and has to be a multiple of 16): d is a multiple of 8, so d / 4 + 1 is odd too.
__host__ __device__ constexpr int tight(int d) { return d + 4; }

// Sizes of a launch, either compile-time constants (the frequent shapes: strides fold into the
// instructions, loops unroll, divisions become shifts) or read from the geometry (everything else).
template <int C_, int DK_, int DV_>
struct FixedDims {
    static constexpr int kC = C_, kDK = DK_, kDV = DV_;      // 0 = not known at compile time
    __device__ explicit FixedDims(const Geom &) {}
    __device__ constexpr int C() const { return C_; }
    __device__ constexpr int dk() const { return DK_; }
    __device__ constexpr int dv() const { return DV_; }
};
struct AnyDims {
    static constexpr int kC = 0, kDK = 0, kDV = 0;
    int c_, dk_, dv_;
    __device__ explicit AnyDims(const Geom &g) : c_(g.C), dk_(g.dk), dv_(g.dv) {}
    __device__ int C() const { return c_; }
    __device__ int dk() const { return dk_; }
    __device__ int dv() const { return dv_; }
};

// Device-side arguments of the value-channel gate (unused by the kernels instantiated without it).
struct BetaDev {
    const float *bgate;     // log(beta) [B][L][H][d_v]
    float *gamma_v;         // [B*H][N][d_v]  exp of the chunk totals of bgate
    float *dbgate;          // gradient with respect to bgate (backward pass)
    float *xtot;            // [B*H][N][d_v]  chunk totals of o*do - v*dv (backward pass)
};

__device__ __forceinline__ float tf32r(float x)
{
    uint32_t u;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
    return __uint_as_float(u);
}

// Rounding of a tile element: none when the operands are split at fragment load (PR).
template <bool PR>
__device__ __forceinline__ float rnd(float x) { return PR ? x : tf32r(x); }
// x = hi + lo with hi the tf32 truncation of x (what the tensor core reads of an fp32 register anyway).
__device__ __forceinline__ void split_tf32(float x, uint32_t &hi, uint32_t &lo)
{
    hi = __float_as_uint(x) & 0xffffe000u;
    lo = __float_as_uint(x - __uint_as_float(hi));
}

__device__ __forceinline__ void mma8(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// One warp: acc[nb] += A(r0 .. r0+15, k) * B(k, c0 + 8 nb .. c0 + 8 nb + 7) for k in [k0, k1), nb < nbw.
// A(m, k) = A[m*sam + k*sak], B(k, n) = Bm[k*sbk + n*sbn]; k0, k1 multiples of 8.
// Fragment layout of m16n8k8: with g = lane / 4, t = lane % 4 a lane holds A(g | g+8, t | t+4),
// B(t | t+4, g) and the results C(g | g+8, 2t | 2t+1).
template <bool PR, int NB>
__device__ __forceinline__ void warp_mma(float (&acc)[NB][4], const float *A, int sam, int sak, int r0,
                                         const float *Bm, int sbk, int sbn, int c0, int nbw, int k0, int k1)
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const float *pa = A + (r0 + g) * sam + (t + k0) * sak;
    const float *pb = Bm + (t + k0) * sbk + (c0 + g) * sbn;
#pragma unroll 2
    for (int k = k0; k < k1; k += 8) {
        const float af[4] = {pa[0], pa[8 * sam], pa[4 * sak], pa[8 * sam + 4 * sak]};
        uint32_t a[4], al[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (PR) split_tf32(af[i], a[i], al[i]);
            else a[i] = __float_as_uint(af[i]);
        }
#pragma unroll
        for (int nb = 0; nb < NB; ++nb)
            if (nb < nbw) {
                const float bf0 = pb[8 * nb * sbn], bf1 = pb[4 * sbk + 8 * nb * sbn];
                if (PR) {
                    uint32_t b0, b1, b0l, b1l;
                    split_tf32(bf0, b0, b0l);
                    split_tf32(bf1, b1, b1l);
                    mma8(acc[nb], al, b0, b1);          // the small terms first
                    mma8(acc[nb], a, b0l, b1l);
                    mma8(acc[nb], a, b0, b1);
                } else {
                    mma8(acc[nb], a, __float_as_uint(bf0), __float_as_uint(bf1));
                }
            }
        pa += 8 * sak;
        pb += 8 * sbk;
    }
}

template <int NB>
__device__ __forceinline__ void zero(float (&acc)[NB][4])
{
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nb][i] = 0.f;
}

// Calls f(row, col, v0, v1) for every pair of adjacent result columns this lane holds (col even).
template <int NB, typename F>
__device__ __forceinline__ void for_pairs(const float (&acc)[NB][4], int r0, int c0, int nbw, F f)
{
    const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb)
        if (nb < nbw) {
            f(r0 + g, c0 + 8 * nb + 2 * t, acc[nb][0], acc[nb][1]);
            f(r0 + g + 8, c0 + 8 * nb + 2 * t, acc[nb][2], acc[nb][3]);
        }
}

// The warp tiles of an M x N result (M a multiple of 16, N of 8): 16 rows by a group of 8-column
// fragments; the columns are split until every warp has a tile (the last group may be shorter).
__host__ __device__ constexpr int tile_splits(int M, int N)
{
    int cs = 1;
    while ((M >> 4) * cs < kWarps && cs < (N >> 3)) cs *= 2;
    return cs;
}
__host__ __device__ constexpr int tile_frags(int M, int N) { return ((N >> 3) + tile_splits(M, N) - 1) / tile_splits(M, N); }
// Fragments per warp tile as a compile-time bound: exact when both extents are known, else the maximum.
__host__ __device__ constexpr int frag_bound(int M, int N) { return (M > 0 && N > 0) ? tile_frags(M, N) : kMaxNB; }
struct Tiling {
    int nrt, nfrag, nbw, ntiles;
    __device__ Tiling(int M, int N) : nrt(M >> 4), nfrag(N >> 3), nbw(tile_frags(M, N)), ntiles((M >> 4) * tile_splits(M, N)) {}
    // first row, first column and fragment count (<= 0: nothing to do) of a tile
    __device__ void at(int tile, int &r0, int &c0, int &nbt) const
    {
        const int rt = tile % nrt, ct = tile / nrt;
        r0 = 16 * rt;
        c0 = 8 * nbw * ct;
        nbt = min(nbw, nfrag - nbw * ct);
    }
};

__device__ __forceinline__ float2 load2(const float *p) { return *reinterpret_cast<const float2 *>(p); }
__device__ __forceinline__ float2 load2(const __nv_bfloat16 *p) { return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(p)); }
__device__ __forceinline__ void store2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16 *p, float a, float b)
{
    *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}

// ---- tile fills -----------------------------------------------------------------------------------
// sRow[j] = index of the chunk's row j among the (token, head) rows of a [B][L][H][.] tensor, or -1 past
// the end of the sequence.  Every later access to global memory goes through this table.
__device__ __forceinline__ void fill_rows(int *sRow, const Geom &g, int C, int b, int h, int chunk)
{
    for (int j = threadIdx.x; j < C; j += kThreads) {
        const int p = chunk * C + j;
        sRow[j] = p < g.L ? (b * g.L + scan_token(p, g.dir, g.gh, g.gw, g.L)) * g.H + h : -1;
    }
}
// Every tile is filled in one phase at the start of a kernel so that a CTA pays the latency of global
// memory once: fp32 sources travel by cp.async (no registers, all copies in flight together), bf16
// sources in register batches of four 8-byte loads per thread.  Rows past the end of the sequence and
// the padding columns become zero.  The values are rescaled / rounded in place afterwards.
__device__ __forceinline__ void cp_async16(float *dst, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void load_rows(float *dst, int ld, const __nv_bfloat16 *src, const int *sRow, int C, int d, int dp)
{
    constexpr int U = 4;
    const int per_row = dp >> 2, n = C * per_row;      // dp: columns to fill (d, or d padded to 16)
    for (int base = threadIdx.x; base < n; base += U * kThreads) {
        uint2 raw[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * kThreads;
            raw[u] = make_uint2(0u, 0u);
            if (idx < n) {
                const int j = idx / per_row, c = (idx - j * per_row) << 2;
                const int row = sRow[j];
                if (row >= 0 && c < d) raw[u] = *reinterpret_cast<const uint2 *>(src + (size_t)row * d + c);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int idx = base + u * kThreads;
            if (idx < n) {
                const int j = idx / per_row, c = (idx - j * per_row) << 2;
                *reinterpret_cast<float4 *>(dst + j * ld + c) =
                    make_float4(__uint_as_float(raw[u].x << 16), __uint_as_float(raw[u].x & 0xffff0000u),
                                __uint_as_float(raw[u].y << 16), __uint_as_float(raw[u].y & 0xffff0000u));
            }
        }
    }
}
__device__ __forceinline__ void load_gates(float *dst, int ld, const float *gate, const int *sRow, int C, int dk, int dp)
{
    const int per_row = dp >> 2;
    for (int idx = threadIdx.x; idx < C * per_row; idx += kThreads) {
        const int j = idx / per_row, c = (idx - j * per_row) << 2;
        const int row = sRow[j];
        if (row >= 0 && c < dk) cp_async16(dst + j * ld + c, gate + (size_t)row * dk + c);
        else *reinterpret_cast<float4 *>(dst + j * ld + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
__device__ __forceinline__ void load_rows(float *dst, int ld, const float *src, const int *sRow, int C, int d, int dp)
{
    load_gates(dst, ld, src, sRow, C, d, dp);       // fp32 rows travel like the gates
}
// A [dk][dv] state of the workspace (rounded to tf32 by the scan kernels) -> [dk][ld] tile.
__device__ __forceinline__ void load_state(float *dst, int ld, const float *src, int dk, int dv)
{
    const int per_row = dv >> 2;
    for (int idx = threadIdx.x; idx < dk * per_row; idx += kThreads) {
        const int r = idx / per_row, c = (idx - r * per_row) << 2;
        if (r < dk && c < dv) cp_async16(dst + r * ld + c, src + r * dv + c);
        else *reinterpret_cast<float4 *>(dst + r * ld + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
}
// In place: gates -> inclusive prefix sums down the rows of the chunk; sLast receives the last row.
// Four threads per channel take a quarter of the rows each; sSeg ([4][dkp]) carries the quarter totals.
// Contains two barriers.
__device__ __forceinline__ void prefix_gates(float *lam, int ld, int C, int dkp, float *sLast, float *sSeg)
{
    const int rows = C >> 2;                    // C is a multiple of 16
    const int c = threadIdx.x % dkp, seg = threadIdx.x / dkp;      // 4 * dkp <= kThreads
    float run = 0.f;
    if (seg < 4) {
#pragma unroll 8
        for (int j = seg * rows; j < (seg + 1) * rows; ++j) {
            run += lam[j * ld + c];
            lam[j * ld + c] = run;
        }
        sSeg[seg * dkp + c] = run;
    }
    __syncthreads();
    if (seg < 4) {
        float add = 0.f;
        for (int sg = 0; sg < seg; ++sg) add += sSeg[sg * dkp + c];
        if (seg > 0) {
#pragma unroll 8
            for (int j = seg * rows; j < (seg + 1) * rows; ++j) lam[j * ld + c] += add;
        }
        if (seg == 3) sLast[c] = run + add;
    }
    __syncthreads();
}
// In place: sQ (raw q) -> Qt = q*exp(Lam), sK (raw k) -> Kt = k*exp(-Lam), or with sLast given
// -> Kh = k*exp(Lam_{C-1}-Lam); rounded to tf32.  Either tile may be null.
template <bool PR>
__device__ __forceinline__ void scale_qk(float *sQ, float *sK, const float *sLam, const float *sLast, int ldk, int C, int dp)
{
    const int per_row = dp >> 2;
    for (int idx = threadIdx.x; idx < C * per_row; idx += kThreads) {
        const int j = idx / per_row, c = (idx - j * per_row) << 2;
        const float4 lam = *reinterpret_cast<const float4 *>(sLam + j * ldk + c);
        if (sQ) {
            const float4 x = *reinterpret_cast<const float4 *>(sQ + j * ldk + c);
            *reinterpret_cast<float4 *>(sQ + j * ldk + c) = make_float4(
                rnd<PR>(x.x * __expf(lam.x)), rnd<PR>(x.y * __expf(lam.y)), rnd<PR>(x.z * __expf(lam.z)), rnd<PR>(x.w * __expf(lam.w)));
        }
        if (sK) {
            float4 e = make_float4(-lam.x, -lam.y, -lam.z, -lam.w);
            if (sLast) {
                const float4 last = *reinterpret_cast<const float4 *>(sLast + c);
                e = make_float4(last.x - lam.x, last.y - lam.y, last.z - lam.z, last.w - lam.w);
            }
            const float4 x = *reinterpret_cast<const float4 *>(sK + j * ldk + c);
            *reinterpret_cast<float4 *>(sK + j * ldk + c) = make_float4(
                rnd<PR>(x.x * __expf(e.x)), rnd<PR>(x.y * __expf(e.y)), rnd<PR>(x.z * __expf(e.z)), rnd<PR>(x.w * __expf(e.w)));
        }
    }
}

// sP[t][s] = A_t . B_s for s <= t, 0 above the diagonal, rounded to tf32 (A, B: [C][ld] tiles, contraction
// over the first K columns).  The diagonal has weight 1: the token's own k^T v enters undecayed.
template <int NB, bool PR>
__device__ __forceinline__ void masked_scores(float *sP, int ldp, const float *A, const float *Bm, int ld, int C, int K)
{
    const Tiling tl(C, C);
    const int warp = threadIdx.x >> 5;
    for (int tile = warp; tile < tl.ntiles; tile += kWarps) {
        int r0, c0, nbt;
        tl.at(tile, r0, c0, nbt);
        if (nbt <= 0) continue;
        float acc[NB][4];
        zero(acc);
        if (c0 <= r0 + 15) warp_mma<PR>(acc, A, ld, 1, r0, Bm, 1, ld, c0, nbt, 0, K);
        for_pairs(acc, r0, c0, nbt, [&](int t, int s, float v0, float v1) {
            *reinterpret_cast<float2 *>(sP + t * ldp + s) = make_float2(s <= t ? rnd<PR>(v0) : 0.f, s + 1 <= t ? rnd<PR>(v1) : 0.f);
        });
    }
}

// ---- kernel 1: chunk-local state contributions ------------------------------------------------------
// U = Kh^T V (and, for the backward pass, W = Qt^T dO); gamma = exp(Lam_{C-1}).
// BETA: with the value-channel gate the value side mirrors the key side: M = prefix sums of log(beta),
// gamma_v = exp(M_{C-1}), U = Kh^T Vh with Vh = v*exp(M_{C-1}-M), W = Qt^T G with G = dO*exp(M).
template <bool BWD, typename DM, bool BETA, typename TI>
__global__ void __launch_bounds__(kThreads)
mma_chunk_state(const TI *__restrict__ q, const TI *__restrict__ k, const TI *__restrict__ v, const float *__restrict__ gate,
                const TI *__restrict__ d_out, float *__restrict__ states, float *__restrict__ gamma,
                float *__restrict__ dstates, BetaDev bd, Geom g)
{
    constexpr bool PR = std::is_same<TI, float>::value;
    extern __shared__ __align__(16) float smem[];
    __shared__ int sRow[128];
    const DM dm(g);
    const int C = dm.C(), dk = dm.dk(), dv = dm.dv();
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int dkp = pad16(dk), dvp = pad16(dv), ldk = pitch(dk), ldv = pitch(dv);
    float *sLam = smem;                     // gates -> Lam
    float *sX = sLam + C * ldk;             // k -> Kh
    float *sV = sX + C * ldk;
    float *sLast = sV + C * ldv;            // [dkp]
    float *sSeg = sLast + dkp;              // [4][dkp]
    float *sQ = sSeg + 4 * dkp;             // BWD: q -> Qt
    float *sG = sQ + (BWD ? C * ldk : 0);   // BWD: dO
    float *sM = sG + (BWD ? C * ldv : 0);   // BETA: log(beta) -> M
    float *sMlast = sM + C * ldv;           // [dvp]
    float *sSegV = sMlast + dvp;            // [4][dvp]

    fill_rows(sRow, g, C, b, h, chunk);
    __syncthreads();
    if (BETA) load_gates(sM, ldv, bd.bgate, sRow, C, dv, dvp);
    load_gates(sLam, ldk, gate, sRow, C, dk, dkp);
    load_rows(sX, ldk, k, sRow, C, dk, dkp);
    load_rows(sV, ldv, v, sRow, C, dv, dvp);
    if (BWD) {
        load_rows(sQ, ldk, q, sRow, C, dk, dkp);
        load_rows(sG, ldv, d_out, sRow, C, dv, dvp);
    }
    cp_async_wait_all();
    __syncthreads();
    prefix_gates(sLam, ldk, C, dkp, sLast, sSeg);
    if (BETA) prefix_gates(sM, ldv, C, dvp, sMlast, sSegV);
    const size_t chunk_id = (size_t)bh * g.N + chunk;
    for (int c = threadIdx.x; c < dk; c += kThreads) gamma[chunk_id * dk + c] = __expf(sLast[c]);
    scale_qk<PR>(BWD ? sQ : nullptr, sX, sLam, sLast, ldk, C, dkp);
    if (BETA) {
        for (int e = threadIdx.x; e < dv; e += kThreads) bd.gamma_v[chunk_id * dv + e] = __expf(sMlast[e]);
        scale_qk<PR>(BWD ? sG : nullptr, sV, sM, sMlast, ldv, C, dvp);      // G = dO*exp(M), Vh = v*exp(M_{C-1}-M)
    }
    __syncthreads();
    constexpr int NB = frag_bound(pad16(DM::kDK), DM::kDV);
    const Tiling tl(dkp, dv);
    const int warp = threadIdx.x >> 5;
    float *U = states + chunk_id * dk * dv;
    float *W = BWD ? dstates + chunk_id * dk * dv : nullptr;
    for (int tile = warp; tile < tl.ntiles; tile += kWarps) {
        int r0, c0, nbt;
        tl.at(tile, r0, c0, nbt);
        if (nbt <= 0) continue;
        float acc[NB][4];
        zero(acc);
        warp_mma<PR>(acc, sX, 1, ldk, r0, sV, ldv, 1, c0, nbt, 0, C);           // sum_t Kh[t][c] V[t][e]
        for_pairs(acc, r0, c0, nbt, [&](int c, int e, float v0, float v1) {
            if (c < dk && e < dv) store2(U + c * dv + e, v0, v1);
        });
        if (BWD) {
            zero(acc);
            warp_mma<PR>(acc, sQ, 1, ldk, r0, sG, ldv, 1, c0, nbt, 0, C);       // sum_t Qt[t][c] dO[t][e]
            for_pairs(acc, r0, c0, nbt, [&](int c, int e, float v0, float v1) {
                if (c < dk && e < dv) store2(W + c * dv + e, v0, v1);
            });
        }
    }
}

// ---- kernel 3: outputs ------------------------------------------------------------------------------
// out = tril(Qt Kt^T) V + Qt S
// BETA: out = exp(M) * (tril(Qt Kt^T) Vt + Qt S) with Vt = v*exp(-M).
template <typename TO, typename DM, bool BETA, typename TI>
__global__ void __launch_bounds__(kThreads)
mma_chunk_out(const TI *__restrict__ q, const TI *__restrict__ k, const TI *__restrict__ v, const float *__restrict__ gate,
              const float *__restrict__ states, TO *__restrict__ out, BetaDev bd, Geom g)
{
    constexpr bool PR = std::is_same<TI, float>::value;
    extern __shared__ __align__(16) float smem[];
    __shared__ int sRow[128];
    const DM dm(g);
    const int C = dm.C(), dk = dm.dk(), dv = dm.dv();
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int dkp = dk, ldk = tight(dk), ldv = tight(dv), ldp = tight(C);      // no padding columns here
    float *sLam = smem;
    float *sQ = sLam + C * ldk;
    float *sK = sQ + C * ldk;
    float *sV = sK + C * ldk;
    float *sS = sV + C * ldv;               // [dkp][ldv]
    float *sLast = sS + dkp * ldv;          // [dkp]
    float *sSeg = sLast + dkp;              // [4][dkp]
    float *sP = (C <= dk) ? sLam : sSeg + 4 * dkp;       // the scores reuse the gate tile when they fit
    float *sM = sSeg + 4 * dkp + (C <= dk ? 0 : C * ldp);   // BETA: log(beta) -> M
    float *sMlast = sM + C * ldv;           // [dv]
    float *sSegV = sMlast + dv;             // [4][dv]

    fill_rows(sRow, g, C, b, h, chunk);
    __syncthreads();
    if (BETA) load_gates(sM, ldv, bd.bgate, sRow, C, dv, dv);
    load_gates(sLam, ldk, gate, sRow, C, dk, dk);
    load_state(sS, ldv, states + ((size_t)bh * g.N + chunk) * dk * dv, dk, dv);
    load_rows(sV, ldv, v, sRow, C, dv, dv);
    load_rows(sQ, ldk, q, sRow, C, dk, dk);
    load_rows(sK, ldk, k, sRow, C, dk, dk);
    cp_async_wait_all();
    __syncthreads();
    prefix_gates(sLam, ldk, C, dkp, sLast, sSeg);
    if (BETA) prefix_gates(sM, ldv, C, dv, sMlast, sSegV);
    scale_qk<PR>(sQ, sK, sLam, nullptr, ldk, C, dk);
    if (BETA) scale_qk<PR>(nullptr, sV, sM, nullptr, ldv, C, dv);           // Vt = v*exp(-M)
    __syncthreads();
    masked_scores<frag_bound(DM::kC, DM::kC), PR>(sP, ldp, sQ, sK, ldk, C, dk);
    __syncthreads();
    constexpr int NB = frag_bound(DM::kC, DM::kDV);
    const Tiling tl(C, dv);
    const int warp = threadIdx.x >> 5;
    for (int tile = warp; tile < tl.ntiles; tile += kWarps) {
        int r0, c0, nbt;
        tl.at(tile, r0, c0, nbt);
        if (nbt <= 0) continue;
        float acc[NB][4];
        zero(acc);
        warp_mma<PR>(acc, sP, ldp, 1, r0, sV, ldv, 1, c0, nbt, 0, r0 + 16);     // columns past the diagonal are zero
        warp_mma<PR>(acc, sQ, ldk, 1, r0, sS, ldv, 1, c0, nbt, 0, dk);
        for_pairs(acc, r0, c0, nbt, [&](int j, int e, float v0, float v1) {
            const int row = sRow[j];
            if (BETA) {
                const float2 m = load2(sM + j * ldv + e);
                v0 *= __expf(m.x);
                v1 *= __expf(m.y);
            }
            if (row >= 0 && e < dv) store2(out + (size_t)row * dv + e, v0, v1);
        });
    }
}

// ---- kernel 4: gradients ----------------------------------------------------------------------------
//   P = tril(Qt Kt^T),  dP = tril(dO V^T)
//   dq = (dP Kt + dO S^T) * exp(Lam)
//   dk = (dP^T Qt + V Dg^T) * exp(-Lam)
//   dv = P^T dO + Kt Dg
//   dgate_j = carry + sum_{r >= j in chunk} (q*dq - k*dk)_r,   q*dq = Qt*(dq accumulator), k*dk alike
// BETA: the same formulas with Vt = v*exp(-M) for V and G = dO*exp(M) for dO (Dg then carries both
// decays); dv = (P^T G + Kt Dg) * exp(-M), and the gradient of log(beta) is, mirroring dgate,
//   dbgate_j = sum_{r >= j} (o*dO - v*dv)_r  with  o*dO = (P Vt + Qt S)*G  and  v*dv = Vt*(dv accumulator)
// (the unscaled output P Vt + Qt S is recomputed here, two more products, rather than read back in
// storage precision), summed here inside the chunk; the chunk total goes to xtot for the cross-chunk part.
template <typename TO, typename DM, bool BETA, typename TI>
__global__ void __launch_bounds__(kThreads)
mma_chunk_bwd(const TI *__restrict__ q, const TI *__restrict__ k, const TI *__restrict__ v, const float *__restrict__ gate,
              const TI *__restrict__ d_out, const float *__restrict__ states,
              const float *__restrict__ dstates, const float *__restrict__ carry, TO *__restrict__ dq,
              TO *__restrict__ dk_out, TO *__restrict__ dv_out, float *__restrict__ dgate, BetaDev bd, Geom g)
{
    constexpr bool PR = std::is_same<TI, float>::value;
    extern __shared__ __align__(16) float smem[];
    __shared__ int sRow[128];
    const DM dm(g);
    const int C = dm.C(), dk = dm.dk(), dv = dm.dv();
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int dkp = dk, ldk = tight(dk), ldv = tight(dv), ldp = tight(C);      // no padding columns here
    float *sLam = smem;                     // Lam, later x = q*dq - k*dk
    float *sQ = sLam + C * ldk;
    float *sK = sQ + C * ldk;
    float *sV = sK + C * ldk;
    float *sG = sV + C * ldv;               // dO
    float *sS = sG + C * ldv;               // [dkp][ldv]
    float *sD = sS + dkp * ldv;             // [dkp][ldv]  Dg, as the scan kernel stores it
    float *sP = sD + dkp * ldv;             // [C][ldp]
    float *sdP = sP + C * ldp;              // [C][ldp]
    float *sLast = sdP + C * ldp;           // [dkp]
    float *sSeg = sLast + dkp;              // [4][dkp]
    float *sM = sSeg + 4 * dkp;             // BETA: log(beta) -> M, later x = o*dO - v*dv
    float *sMlast = sM + C * ldv;           // [dv]
    float *sSegV = sMlast + dv;             // [4][dv]
    const size_t chunk_id = (size_t)bh * g.N + chunk;

    fill_rows(sRow, g, C, b, h, chunk);
    __syncthreads();
    if (BETA) load_gates(sM, ldv, bd.bgate, sRow, C, dv, dv);
    load_gates(sLam, ldk, gate, sRow, C, dk, dk);
    load_state(sS, ldv, states + chunk_id * dk * dv, dk, dv);
    load_state(sD, ldv, dstates + chunk_id * dk * dv, dk, dv);
    load_rows(sV, ldv, v, sRow, C, dv, dv);
    load_rows(sG, ldv, d_out, sRow, C, dv, dv);
    load_rows(sQ, ldk, q, sRow, C, dk, dk);
    load_rows(sK, ldk, k, sRow, C, dk, dk);
    cp_async_wait_all();
    __syncthreads();
    prefix_gates(sLam, ldk, C, dkp, sLast, sSeg);
    if (BETA) prefix_gates(sM, ldv, C, dv, sMlast, sSegV);
    scale_qk<PR>(sQ, sK, sLam, nullptr, ldk, C, dk);
    if (BETA) scale_qk<PR>(sG, sV, sM, nullptr, ldv, C, dv);                // G = dO*exp(M), Vt = v*exp(-M)
    __syncthreads();
    masked_scores<frag_bound(DM::kC, DM::kC), PR>(sP, ldp, sQ, sK, ldk, C, dk);
    masked_scores<frag_bound(DM::kC, DM::kC), PR>(sdP, ldp, sG, sV, ldv, C, dv);
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gi = lane >> 2, ti = lane & 3;
    {
        // dv[s][e] = sum_{t >= s} P[t][s] dO[t][e] + sum_c Kt[s][c] Dg[c][e]
        constexpr int NB = frag_bound(DM::kC, DM::kDV);
        const Tiling tl(C, dv);
        for (int tile = warp; tile < tl.ntiles; tile += kWarps) {
            int r0, c0, nbt;
            tl.at(tile, r0, c0, nbt);
            if (nbt <= 0) continue;
            float acc[NB][4];
            zero(acc);
            warp_mma<PR>(acc, sP, 1, ldp, r0, sG, ldv, 1, c0, nbt, r0, C);
            warp_mma<PR>(acc, sK, ldk, 1, r0, sD, ldv, 1, c0, nbt, 0, dk);
            if (BETA) {
                // unscaled output of the same tile, then x = o*dO - v*dv = (P Vt + Qt S)*G - Vt*(dv accumulator)
                float oh[NB][4];
                zero(oh);
                warp_mma<PR>(oh, sP, ldp, 1, r0, sV, ldv, 1, c0, nbt, 0, r0 + 16);
                warp_mma<PR>(oh, sQ, ldk, 1, r0, sS, ldv, 1, c0, nbt, 0, dk);
#pragma unroll
                for (int nb = 0; nb < NB; ++nb)
                    if (nb < nbt) {
#pragma unroll
                        for (int i = 0; i < 4; i += 2) {
                            const int off = (r0 + gi + 4 * i) * ldv + c0 + 8 * nb + 2 * ti;
                            const float2 vt = load2(sV + off), gg = load2(sG + off);
                            oh[nb][i] = oh[nb][i] * gg.x - vt.x * acc[nb][i];
                            oh[nb][i + 1] = oh[nb][i + 1] * gg.y - vt.y * acc[nb][i + 1];
                        }
                    }
                // this thread alone touches its elements of M: scale dv by exp(-M), then leave x there
                for_pairs(acc, r0, c0, nbt, [&](int j, int e, float v0, float v1) {
                    const int row = sRow[j];
                    const float2 m = load2(sM + j * ldv + e);
                    if (row >= 0 && e < dv) store2(dv_out + (size_t)row * dv + e, v0 * __expf(-m.x), v1 * __expf(-m.y));
                });
                __syncwarp();
                for_pairs(oh, r0, c0, nbt, [&](int j, int e, float v0, float v1) {
                    *reinterpret_cast<float2 *>(sM + j * ldv + e) = make_float2(v0, v1);
                });
            } else {
                for_pairs(acc, r0, c0, nbt, [&](int j, int e, float v0, float v1) {
                    const int row = sRow[j];
                    if (row >= 0 && e < dv) store2(dv_out + (size_t)row * dv + e, v0, v1);
                });
            }
        }
    }
    {
        // dq and dk of the same (row, channel) tile; x = q*dq - k*dk replaces Lam, element by element
        constexpr int NB = frag_bound(DM::kC, DM::kDK);
        const Tiling tl(C, dk);
        for (int tile = warp; tile < tl.ntiles; tile += kWarps) {
            int r0, c0, nbt;
            tl.at(tile, r0, c0, nbt);
            if (nbt <= 0) continue;
            float acc[NB][4], xq[NB][4];
            zero(acc);
            warp_mma<PR>(acc, sdP, ldp, 1, r0, sK, ldk, 1, c0, nbt, 0, r0 + 16);          // sum_{s <= t} dP[t][s] Kt[s][c]
            warp_mma<PR>(acc, sG, ldv, 1, r0, sS, 1, ldv, c0, nbt, 0, dv);                // sum_e dO[t][e] S[c][e]
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
                if (nb < nbt) {
#pragma unroll
                    for (int i = 0; i < 4; i += 2) {
                        const float2 qt = *reinterpret_cast<const float2 *>(sQ + (r0 + gi + 4 * i) * ldk + c0 + 8 * nb + 2 * ti);
                        xq[nb][i] = qt.x * acc[nb][i];
                        xq[nb][i + 1] = qt.y * acc[nb][i + 1];
                    }
                }
            for_pairs(acc, r0, c0, nbt, [&](int j, int c, float v0, float v1) {
                const int row = sRow[j];
                if (row >= 0 && c < dk) {
                    const float2 lam = *reinterpret_cast<const float2 *>(sLam + j * ldk + c);
                    store2(dq + (size_t)row * dk + c, v0 * __expf(lam.x), v1 * __expf(lam.y));
                }
            });
            zero(acc);
            warp_mma<PR>(acc, sdP, 1, ldp, r0, sQ, ldk, 1, c0, nbt, r0, C);               // sum_{t >= s} dP[t][s] Qt[t][c]
            warp_mma<PR>(acc, sV, ldv, 1, r0, sD, 1, ldv, c0, nbt, 0, dv);                // sum_e V[s][e] Dg[c][e]
#pragma unroll
            for (int nb = 0; nb < NB; ++nb)
                if (nb < nbt) {
#pragma unroll
                    for (int i = 0; i < 4; i += 2) {
                        const float2 kt = *reinterpret_cast<const float2 *>(sK + (r0 + gi + 4 * i) * ldk + c0 + 8 * nb + 2 * ti);
                        xq[nb][i] -= kt.x * acc[nb][i];
                        xq[nb][i + 1] -= kt.y * acc[nb][i + 1];
                    }
                }
            for_pairs(acc, r0, c0, nbt, [&](int j, int c, float v0, float v1) {
                const int row = sRow[j];
                if (row >= 0 && c < dk) {
                    const float2 lam = *reinterpret_cast<const float2 *>(sLam + j * ldk + c);
                    store2(dk_out + (size_t)row * dk + c, v0 * __expf(-lam.x), v1 * __expf(-lam.y));
                }
            });
            __syncwarp();
            for_pairs(xq, r0, c0, nbt, [&](int j, int c, float v0, float v1) {
                *reinterpret_cast<float2 *>(sLam + j * ldk + c) = make_float2(v0, v1);
            });
        }
    }
    __syncthreads();
    // gate gradient: suffix sums of x down the chunk plus what later chunks carry in; four threads per
    // channel take a quarter of the rows each
    {
        const int rows = C >> 2;
        const int c = threadIdx.x % dkp, seg = threadIdx.x / dkp;
        float run = 0.f;
        if (seg < 4) {
#pragma unroll 8
            for (int j = (seg + 1) * rows - 1; j >= seg * rows; --j) {
                run += sLam[j * ldk + c];
                sLam[j * ldk + c] = run;
            }
            sSeg[seg * dkp + c] = run;
        }
        // the value-channel gate: the same inside the chunk, without the carry (added by a later pass)
        const int cv = threadIdx.x % dv, segv = threadIdx.x / dv;
        if (BETA && segv < 4) {
            float runv = 0.f;
#pragma unroll 8
            for (int j = (segv + 1) * rows - 1; j >= segv * rows; --j) {
                runv += sM[j * ldv + cv];
                sM[j * ldv + cv] = runv;
            }
            sSegV[segv * dv + cv] = runv;
        }
        __syncthreads();
        if (seg < 4 && c < dk) {
            float add = carry[chunk_id * dk + c];
            for (int sg = seg + 1; sg < 4; ++sg) add += sSeg[sg * dkp + c];
            for (int j = seg * rows; j < (seg + 1) * rows; ++j) {
                const int row = sRow[j];
                if (row >= 0) dgate[(size_t)row * dk + c] = sLam[j * ldk + c] + add;
            }
        }
        if (BETA && segv < 4) {
            float add = 0.f;
            for (int sg = segv + 1; sg < 4; ++sg) add += sSegV[sg * dv + cv];
            for (int j = segv * rows; j < (segv + 1) * rows; ++j) {
                const int row = sRow[j];
                if (row >= 0) bd.dbgate[(size_t)row * dv + cv] = sM[j * ldv + cv] + add;
            }
            if (segv == 0) bd.xtot[chunk_id * dv + cv] = sSegV[cv] + add;
        }
    }
}

size_t smem_state(const Geom &g, bool bwd, bool beta)
{
    size_t n = (size_t)g.C * (pitch(g.dk) * (bwd ? 3 : 2) + pitch(g.dv) * (bwd ? 2 : 1)) + 5 * pad16(g.dk);
    if (beta) n += (size_t)g.C * pitch(g.dv) + 5 * pad16(g.dv);
    return sizeof(float) * n;
}
size_t smem_out(const Geom &g, bool beta)
{
    size_t n = (size_t)g.C * (3 * tight(g.dk) + tight(g.dv)) + (size_t)g.dk * tight(g.dv) + 5 * g.dk;
    if (g.C > g.dk) n += (size_t)g.C * tight(g.C);
    if (beta) n += (size_t)g.C * tight(g.dv) + 5 * g.dv;
    return sizeof(float) * n;
}
size_t smem_bwd(const Geom &g, bool beta)
{
    size_t n = (size_t)g.C * (3 * tight(g.dk) + 2 * tight(g.dv) + 2 * tight(g.C)) + 2 * (size_t)g.dk * tight(g.dv) + 5 * g.dk;
    if (beta) n += (size_t)g.C * tight(g.dv) + 5 * g.dv;
    return sizeof(float) * n;
}
constexpr size_t kMaxSmem = 227 * 1024 - 1024;      // the row table is static shared memory

template <typename K>
dig_status set_smem(K kernel, size_t bytes)
{
    if (bytes > kMaxSmem) return DIG_ERR_UNSUPPORTED;
    return ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), bytes);
}

// The value-channel gate keeps two more blocks behind the common workspace: gamma_v and, for the
// backward pass, the chunk totals of o*do - v*dv, both [B*H][N][d_v].
size_t beta_block(const Geom &g) { return align256((size_t)g.B * g.H * g.N * g.dv * sizeof(float)); }
BetaDev beta_dev(const GlaArgs &a, const Workspace &w, bool backward)
{
    BetaDev bd{};
    if (a.bio.bgate == nullptr) return bd;
    char *p = reinterpret_cast<char *>(a.ws) + w.bytes;
    bd.bgate = a.bio.bgate;
    bd.gamma_v = reinterpret_cast<float *>(p);
    if (backward) {
        bd.dbgate = a.bio.dbgate;
        bd.xtot = reinterpret_cast<float *>(p + beta_block(a.g));
    }
    return bd;
}

template <typename TO, typename DM, bool BETA, typename TI = bf16>
dig_status fwd_dims(const GlaArgs &a)
{
    constexpr bool kRound = !std::is_same<TI, float>::value;     // states rounded to tf32 by the scans
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, false);
    const BetaDev bd = beta_dev(a, w, false);
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = mma_chunk_state<false, DM, BETA, TI>;
    if ((st = set_smem(k1, smem_state(g, false, BETA))) != DIG_OK) return st;
    auto k3 = mma_chunk_out<TO, DM, BETA, TI>;
    if ((st = set_smem(k3, smem_out(g, BETA))) != DIG_OK) return st;
    {
        KernelTimer t(KID_MMA_STATE, a.stream);
        k1<<<grid, kThreads, smem_state(g, false, BETA), a.stream>>>((const TI *)a.q, (const TI *)a.k, (const TI *)a.v,
                                                                    a.gate, nullptr, w.states, w.gamma, nullptr, bd, g);
    }
    if (BETA) st = launch_state_scan_fwd_beta(w, bd.gamma_v, g, a.stream, kRound);
    else st = launch_state_scan_fwd(w, g, a.stream, a.sio, kRound);
    if (st != DIG_OK) return st;
    KernelTimer t(KID_MMA_OUT, a.stream);
    k3<<<grid, kThreads, smem_out(g, BETA), a.stream>>>((const TI *)a.q, (const TI *)a.k, (const TI *)a.v, a.gate,
                                                        w.states, (TO *)a.out, bd, g);
    return cuda_ok(cudaGetLastError());
}

template <typename TO, typename DM, bool BETA, typename TI = bf16>
dig_status bwd_dims(const GlaArgs &a)
{
    constexpr bool kRound = !std::is_same<TI, float>::value;
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, true);
    const BetaDev bd = beta_dev(a, w, true);
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = mma_chunk_state<true, DM, BETA, TI>;
    if ((st = set_smem(k1, smem_state(g, true, BETA))) != DIG_OK) return st;
    auto k4 = mma_chunk_bwd<TO, DM, BETA, TI>;
    if ((st = set_smem(k4, smem_bwd(g, BETA))) != DIG_OK) return st;
    {
        KernelTimer t(KID_MMA_STATE, a.stream);
        k1<<<grid, kThreads, smem_state(g, true, BETA), a.stream>>>((const TI *)a.q, (const TI *)a.k, (const TI *)a.v,
                                                                   a.gate, (const TI *)a.d_out, w.states, w.gamma, w.dstates,
                                                                   bd, g);
    }
    if (BETA) {
        if ((st = launch_state_scan_fwd_beta(w, bd.gamma_v, g, a.stream, kRound)) != DIG_OK) return st;
        if ((st = launch_state_scan_bwd_beta(w, bd.gamma_v, g, a.stream, kRound)) != DIG_OK) return st;
    } else {
        if ((st = launch_state_scan_fwd(w, g, a.stream, a.sio, kRound)) != DIG_OK) return st;
        if ((st = launch_state_scan_bwd(w, g, a.stream, a.sio, kRound)) != DIG_OK) return st;
    }
    {
        KernelTimer t(KID_MMA_BWD, a.stream);
        k4<<<grid, kThreads, smem_bwd(g, BETA), a.stream>>>((const TI *)a.q, (const TI *)a.k, (const TI *)a.v, a.gate,
                                                            (const TI *)a.d_out, w.states, w.dstates, w.carry, (TO *)a.dq,
                                                            (TO *)a.dk, (TO *)a.dv, a.dgate, bd, g);
    }
    if (cudaGetLastError() != cudaSuccess) return DIG_ERR_CUDA;
    if (BETA) return launch_beta_carry(bd.dbgate, bd.xtot, g, a.stream);
    return DIG_OK;
}

// The shapes of the paper's models that the tcgen05 family leaves to this one get kernels with
// compile-time sizes: 72-wide heads with 64-token chunks, 64-wide heads with 32-token chunks.
template <typename TO, bool BETA>
dig_status fwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    if (g.C == 64 && g.dk == 72 && g.dv == 72) return fwd_dims<TO, FixedDims<64, 72, 72>, BETA>(a);
    if (!BETA && g.C == 32 && g.dk == 64 && g.dv == 64) return fwd_dims<TO, FixedDims<32, 64, 64>, false>(a);
    if (BETA && g.C == 64 && g.dk == 64 && g.dv == 64) return fwd_dims<TO, FixedDims<64, 64, 64>, true>(a);
    return fwd_dims<TO, AnyDims, BETA>(a);
}
template <typename TO, bool BETA>
dig_status bwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    if (g.C == 64 && g.dk == 72 && g.dv == 72) return bwd_dims<TO, FixedDims<64, 72, 72>, BETA>(a);
    if (!BETA && g.C == 32 && g.dk == 64 && g.dv == 64) return bwd_dims<TO, FixedDims<32, 64, 64>, false>(a);
    if (BETA && g.C == 64 && g.dk == 64 && g.dv == 64) return bwd_dims<TO, FixedDims<64, 64, 64>, true>(a);
    return bwd_dims<TO, AnyDims, BETA>(a);
}

}  // namespace

bool mma_supports(int dk, int dv, int chunk, int dtype, bool backward, bool beta)
{
    if (dtype == DIG_F32 && !beta) return false;      // fp32 storage: only the full gate is served here (split operands)
    Geom g{};
    g.dk = dk; g.dv = dv; g.C = chunk;
    if (backward) return smem_bwd(g, beta) <= kMaxSmem && smem_state(g, true, beta) <= kMaxSmem;
    return smem_out(g, beta) <= kMaxSmem && smem_state(g, false, beta) <= kMaxSmem;
}

size_t mma_beta_workspace_bytes(const Geom &g, bool backward)
{
    return carve_workspace(nullptr, g, backward).bytes + beta_block(g) * (backward ? 2 : 1);
}

dig_status mma_gla_fwd(const GlaArgs &a)
{
    const bool beta = a.bio.bgate != nullptr;
    if (a.dtype == DIG_BF16) return beta ? fwd_typed<__nv_bfloat16, true>(a) : fwd_typed<__nv_bfloat16, false>(a);
    if (a.dtype == DIG_BF16_F32OUT) return beta ? fwd_typed<float, true>(a) : fwd_typed<float, false>(a);
    if (a.dtype == DIG_F32 && beta) return fwd_dims<float, AnyDims, true, float>(a);
    return DIG_ERR_UNSUPPORTED;
}

dig_status mma_gla_bwd(const GlaArgs &a)
{
    const bool beta = a.bio.bgate != nullptr;
    if (a.dtype == DIG_BF16) return beta ? bwd_typed<__nv_bfloat16, true>(a) : bwd_typed<__nv_bfloat16, false>(a);
    if (a.dtype == DIG_BF16_F32OUT) return beta ? bwd_typed<float, true>(a) : bwd_typed<float, false>(a);
    if (a.dtype == DIG_F32 && beta) return bwd_dims<float, AnyDims, true, float>(a);
    return DIG_ERR_UNSUPPORTED;
}

}  // namespace dig
