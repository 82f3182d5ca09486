// fp32-FMA kernel family for chunkwise gated linear attention (Eq. attn_gla, evaluated chunk
// by chunk as Section 3.5 describes).  Serves DIG_F32 (products must be fp32-accurate, which a
// single tf32 tensor-core pass is not) and any bf16 request the tensor-core family does not
// cover.  One CTA per (chunk, batch*head); every contraction is a register-blocked 4x4 FMA loop
// over shared-memory tiles.
//
// Notation per chunk (rows j = 0..C-1 in scan order, zero rows past the end of the sequence):
//   Lam_j = inclusive prefix sum of the gates, gamma = exp(Lam_{C-1}),
//   Qt = q*exp(Lam), Kt = k*exp(-Lam), Kh = k*exp(Lam_{C-1}-Lam) = Kt*gamma,
//   S = state entering the chunk, D = dL/d(state leaving the chunk).
#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int kThreads = 256;

// ---- 4x4 register-blocked contractions over shared memory --------------------------------
// acc[i][j] += sum_k A[(r0+i)*lda + k] * Bm[(c0 + j*cstep)*ldb + k]
__device__ __forceinline__ void mm_nt(float (&acc)[4][4], const float *A, int lda, int r0,
                                      const float *Bm, int ldb, int c0, int cstep, int K)
{
    for (int k = 0; k < K; k += 4) {
        float4 a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4 *>(A + (r0 + i) * lda + k);
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const float4 *>(Bm + (c0 + j * cstep) * ldb + k);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j)
                acc[i][j] += a[i].x * b[j].x + a[i].y * b[j].y + a[i].z * b[j].z + a[i].w * b[j].w;
    }
}
// acc[i][j] += sum_{k<K} A[(r0+i)*lda + k] * Bm[k*ldb + c0 + j]
__device__ __forceinline__ void mm_nn(float (&acc)[4][4], const float *A, int lda, int r0,
                                      const float *Bm, int ldb, int c0, int K)
{
    for (int k = 0; k < K; k += 4) {
        float4 a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4 *>(A + (r0 + i) * lda + k);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) b[kk] = *reinterpret_cast<const float4 *>(Bm + (k + kk) * ldb + c0);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[i][0] += a[i].x * b[0].x + a[i].y * b[1].x + a[i].z * b[2].x + a[i].w * b[3].x;
            acc[i][1] += a[i].x * b[0].y + a[i].y * b[1].y + a[i].z * b[2].y + a[i].w * b[3].y;
            acc[i][2] += a[i].x * b[0].z + a[i].y * b[1].z + a[i].z * b[2].z + a[i].w * b[3].z;
            acc[i][3] += a[i].x * b[0].w + a[i].y * b[1].w + a[i].z * b[2].w + a[i].w * b[3].w;
        }
    }
}
// acc[i][j] += sum_{k<K} A[k*lda + r0 + i] * Bm[k*ldb + c0 + j]
__device__ __forceinline__ void mm_tn(float (&acc)[4][4], const float *A, int lda, int r0,
                                      const float *Bm, int ldb, int c0, int K)
{
    for (int k = 0; k < K; ++k) {
        const float4 a = *reinterpret_cast<const float4 *>(A + k * lda + r0);
        const float4 b = *reinterpret_cast<const float4 *>(Bm + k * ldb + c0);
        const float av[4] = {a.x, a.y, a.z, a.w};
        const float bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] += av[i] * bv[j];
    }
}
__device__ __forceinline__ void zero(float (&acc)[4][4])
{
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
}

// ---- tile loaders ----------------------------------------------------------------------------
// Copies the chunk's rows of a [B][L][H][d] tensor into shared memory (row stride ld floats),
// rows past the end of the sequence become zero.
template <typename T>
__device__ __forceinline__ void load_tile(float *dst, int ld, const T *src, const Geom &g, int b,
                                          int h, int chunk, int d)
{
    const int per_row = d >> 2;
    for (int idx = threadIdx.x; idx < g.C * per_row; idx += kThreads) {
        const int j = idx / per_row, c = (idx - j * per_row) << 2;
        const int p = chunk * g.C + j;
        float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p < g.L) {
            const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
            val = load4(src + tok_offset(g, b, t, h, d) + c);
        }
        *reinterpret_cast<float4 *>(dst + j * ld + c) = val;
    }
}

// In place: gates -> inclusive prefix sums along the rows of the chunk, one thread per channel.
__device__ __forceinline__ void prefix_gates(float *lam, int ld, int C, int dk)
{
    for (int c = threadIdx.x; c < dk; c += kThreads) {
        float run = 0.f;
        for (int j = 0; j < C; ++j) {
            run += lam[j * ld + c];
            lam[j * ld + c] = run;
        }
    }
}

// ---- kernel 1: chunk-local state contributions ------------------------------------------------
// U = Kh^T V  (and, for the backward pass, W = Qt^T dO); gamma = exp(Lam_{C-1}).
template <typename T, bool BWD>
__global__ void __launch_bounds__(kThreads)
fma_chunk_state(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
                const float *__restrict__ gate, const T *__restrict__ d_out,
                float *__restrict__ states, float *__restrict__ gamma, float *__restrict__ dstates,
                Geom g)
{
    extern __shared__ __align__(16) float smem[];
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int ldk = g.dk + 4, ldv = g.dv + 4;
    float *sX = smem;                       // gates -> Lam -> Kh
    float *sV = sX + g.C * ldk;
    float *sQ = sV + g.C * ldv;             // BWD: Qt
    float *sG = sQ + (BWD ? g.C * ldk : 0); // BWD: dO

    load_tile(sX, ldk, gate, g, b, h, chunk, g.dk);
    load_tile(sV, ldv, v, g, b, h, chunk, g.dv);
    if (BWD) load_tile(sG, ldv, d_out, g, b, h, chunk, g.dv);
    __syncthreads();
    prefix_gates(sX, ldk, g.C, g.dk);
    __syncthreads();
    const size_t chunk_id = (size_t)bh * g.N + chunk;
    for (int c = threadIdx.x; c < g.dk; c += kThreads)
        gamma[chunk_id * g.dk + c] = expf(sX[(g.C - 1) * ldk + c]);
    {
        const int per_row = g.dk >> 2;
        for (int idx = threadIdx.x; idx < g.C * per_row; idx += kThreads) {
            const int j = idx / per_row, c = (idx - j * per_row) << 2;
            const int p = chunk * g.C + j;
            float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), qq = kk;
            if (p < g.L) {
                const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
                kk = load4(k + tok_offset(g, b, t, h, g.dk) + c);
                if (BWD) qq = load4(q + tok_offset(g, b, t, h, g.dk) + c);
            }
            const float4 lam = *reinterpret_cast<const float4 *>(sX + j * ldk + c);
            const float4 last = *reinterpret_cast<const float4 *>(sX + (g.C - 1) * ldk + c);
            if (BWD) {
                *reinterpret_cast<float4 *>(sQ + j * ldk + c) =
                    make_float4(qq.x * expf(lam.x), qq.y * expf(lam.y), qq.z * expf(lam.z), qq.w * expf(lam.w));
            }
            // the last row is read by other threads as `last`: defer its overwrite
            if (j != g.C - 1)
                *reinterpret_cast<float4 *>(sX + j * ldk + c) =
                    make_float4(kk.x * expf(last.x - lam.x), kk.y * expf(last.y - lam.y),
                                kk.z * expf(last.z - lam.z), kk.w * expf(last.w - lam.w));
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < per_row; idx += kThreads) {   // last row: Kh = k
            const int j = g.C - 1, c = idx << 2;
            const int p = chunk * g.C + j;
            float4 kk = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p < g.L) {
                const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
                kk = load4(k + tok_offset(g, b, t, h, g.dk) + c);
            }
            *reinterpret_cast<float4 *>(sX + j * ldk + c) = kk;
        }
    }
    __syncthreads();
    const int nrb = g.dk >> 2, ncb = g.dv >> 2;
    float *U = states + chunk_id * g.dk * g.dv;
    float *W = BWD ? dstates + chunk_id * g.dk * g.dv : nullptr;
    for (int blk = threadIdx.x; blk < nrb * ncb; blk += kThreads) {
        const int r0 = (blk / ncb) << 2, c0 = (blk % ncb) << 2;
        float acc[4][4];
        zero(acc);
        mm_tn(acc, sX, ldk, r0, sV, ldv, c0, g.C);
#pragma unroll
        for (int i = 0; i < 4; ++i)
            *reinterpret_cast<float4 *>(U + (r0 + i) * g.dv + c0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        if (BWD) {
            zero(acc);
            mm_tn(acc, sQ, ldk, r0, sG, ldv, c0, g.C);
#pragma unroll
            for (int i = 0; i < 4; ++i)
                *reinterpret_cast<float4 *>(W + (r0 + i) * g.dv + c0) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        }
    }
}

// Fills sQ = Qt, sK = Kt from the prefix sums held in sLam (sLam is kept).
template <typename T>
__device__ __forceinline__ void make_qt_kt(float *sQ, float *sK, const float *sLam, int ldk,
                                           const T *q, const T *k, const Geom &g, int b, int h,
                                           int chunk)
{
    const int per_row = g.dk >> 2;
    for (int idx = threadIdx.x; idx < g.C * per_row; idx += kThreads) {
        const int j = idx / per_row, c = (idx - j * per_row) << 2;
        const int p = chunk * g.C + j;
        float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), qq = kk;
        if (p < g.L) {
            const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
            const size_t off = tok_offset(g, b, t, h, g.dk) + c;
            kk = load4(k + off);
            qq = load4(q + off);
        }
        const float4 lam = *reinterpret_cast<const float4 *>(sLam + j * ldk + c);
        *reinterpret_cast<float4 *>(sQ + j * ldk + c) =
            make_float4(qq.x * expf(lam.x), qq.y * expf(lam.y), qq.z * expf(lam.z), qq.w * expf(lam.w));
        *reinterpret_cast<float4 *>(sK + j * ldk + c) =
            make_float4(kk.x * expf(-lam.x), kk.y * expf(-lam.y), kk.z * expf(-lam.z), kk.w * expf(-lam.w));
    }
}

// P[t][s] = Qt_t . Kt_s for s <= t, 0 above the diagonal (the token's own k^T v enters undecayed,
// so the diagonal weight is exactly q_t . k_t).
__device__ __forceinline__ void make_masked_scores(float *sP, int ldp, const float *sA, int lda,
                                                   const float *sB, int ldb, int C, int K)
{
    const int nb = C >> 2;
    for (int blk = threadIdx.x; blk < nb * nb; blk += kThreads) {
        const int r0 = (blk / nb) << 2, cb = blk % nb;       // columns cb, cb+nb, cb+2nb, cb+3nb
        float acc[4][4];
        zero(acc);
        if (cb <= r0 + 3) mm_nt(acc, sA, lda, r0, sB, ldb, cb, nb, K);
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int s = cb + j * nb;
                sP[(r0 + i) * ldp + s] = (s <= r0 + i) ? acc[i][j] : 0.f;
            }
    }
}

// ---- kernel 3: outputs ---------------------------------------------------------------------------
// out = tril(Qt Kt^T) V + Qt S
template <typename T, typename TO>
__global__ void __launch_bounds__(kThreads)
fma_chunk_out(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
              const float *__restrict__ gate, const float *__restrict__ states,
              TO *__restrict__ out, Geom g)
{
    extern __shared__ __align__(16) float smem[];
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int ldk = g.dk + 4, ldv = g.dv + 4, ldp = g.C + 4;
    float *sLam = smem;
    float *sQ = sLam + g.C * ldk;
    float *sK = sQ + g.C * ldk;
    float *sV = sK + g.C * ldk;
    float *sS = sV + g.C * ldv;             // [dk][ldv]
    float *sP = sLam;                       // scores reuse the gate buffer once Qt, Kt exist
    // (sP needs C*(C+4) <= C*(dk+4) floats only when C <= dk; otherwise it gets its own space)
    if (g.C > g.dk) sP = sS + g.dk * ldv;

    load_tile(sLam, ldk, gate, g, b, h, chunk, g.dk);
    load_tile(sV, ldv, v, g, b, h, chunk, g.dv);
    {
        const float *S = states + ((size_t)bh * g.N + chunk) * g.dk * g.dv;
        const int per_row = g.dv >> 2;
        for (int idx = threadIdx.x; idx < g.dk * per_row; idx += kThreads) {
            const int r = idx / per_row, c = (idx - r * per_row) << 2;
            *reinterpret_cast<float4 *>(sS + r * ldv + c) = *reinterpret_cast<const float4 *>(S + r * g.dv + c);
        }
    }
    __syncthreads();
    prefix_gates(sLam, ldk, g.C, g.dk);
    __syncthreads();
    make_qt_kt(sQ, sK, sLam, ldk, q, k, g, b, h, chunk);
    __syncthreads();
    make_masked_scores(sP, ldp, sQ, ldk, sK, ldk, g.C, g.dk);
    __syncthreads();
    const int nrb = g.C >> 2, ncb = g.dv >> 2;
    for (int blk = threadIdx.x; blk < nrb * ncb; blk += kThreads) {
        const int r0 = (blk / ncb) << 2, c0 = (blk % ncb) << 2;
        float acc[4][4];
        zero(acc);
        mm_nn(acc, sP, ldp, r0, sV, ldv, c0, r0 + 4);       // columns beyond the diagonal are zero
        mm_nn(acc, sQ, ldk, r0, sS, ldv, c0, g.dk);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int p = chunk * g.C + r0 + i;
            if (p < g.L) {
                const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
                store4(out + tok_offset(g, b, t, h, g.dv) + c0, make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]));
            }
        }
    }
}

// ---- kernel 4: gradients ---------------------------------------------------------------------------
//   dP = tril(dO V^T)
//   dq = (dP Kt + dO S^T) * exp(Lam)
//   dk = (dP^T Qt) * exp(-Lam) + (V D^T) * exp(Lam_{C-1}-Lam)
//   dv = P^T dO + Kh D
//   dgate_j = carry + sum_{r >= j in chunk} (q*dq - k*dk)_r
template <typename T, typename TO>
__global__ void __launch_bounds__(kThreads)
fma_chunk_bwd(const T *__restrict__ q, const T *__restrict__ k, const T *__restrict__ v,
              const float *__restrict__ gate, const T *__restrict__ d_out,
              const float *__restrict__ states, const float *__restrict__ dstates,
              const float *__restrict__ carry, TO *__restrict__ dq, TO *__restrict__ dk,
              TO *__restrict__ dv, float *__restrict__ dgate, Geom g)
{
    extern __shared__ __align__(16) float smem[];
    const int chunk = blockIdx.x, bh = blockIdx.y, b = bh / g.H, h = bh - b * g.H;
    const int ldk = g.dk + 4, ldv = g.dv + 4, ldp = g.C + 4;
    float *sLam = smem;
    float *sQ = sLam + g.C * ldk;
    float *sK = sQ + g.C * ldk;
    float *sV = sK + g.C * ldk;
    float *sG = sV + g.C * ldv;             // dO
    float *sS = sG + g.C * ldv;             // [dk][ldv]
    float *sD = sS + g.dk * ldv;            // [dk][ldv]
    float *sP = sD + g.dk * ldv;            // [C][ldp]
    float *sdP = sP + g.C * ldp;            // [C][ldp]
    float *sX = sdP + g.C * ldp;            // [C][ldk]  q*dq - k*dk

    load_tile(sLam, ldk, gate, g, b, h, chunk, g.dk);
    load_tile(sV, ldv, v, g, b, h, chunk, g.dv);
    load_tile(sG, ldv, d_out, g, b, h, chunk, g.dv);
    {
        const size_t off = ((size_t)bh * g.N + chunk) * g.dk * g.dv;
        const int per_row = g.dv >> 2;
        for (int idx = threadIdx.x; idx < g.dk * per_row; idx += kThreads) {
            const int r = idx / per_row, c = (idx - r * per_row) << 2;
            *reinterpret_cast<float4 *>(sS + r * ldv + c) = *reinterpret_cast<const float4 *>(states + off + r * g.dv + c);
            *reinterpret_cast<float4 *>(sD + r * ldv + c) = *reinterpret_cast<const float4 *>(dstates + off + r * g.dv + c);
        }
    }
    __syncthreads();
    prefix_gates(sLam, ldk, g.C, g.dk);
    __syncthreads();
    make_qt_kt(sQ, sK, sLam, ldk, q, k, g, b, h, chunk);
    __syncthreads();
    make_masked_scores(sP, ldp, sQ, ldk, sK, ldk, g.C, g.dk);
    make_masked_scores(sdP, ldp, sG, ldv, sV, ldv, g.C, g.dv);
    __syncthreads();

    // dv = P^T dO + (Kt*gamma) D
    {
        const int nrb = g.C >> 2, ncb = g.dv >> 2;
        for (int blk = threadIdx.x; blk < nrb * ncb; blk += kThreads) {
            const int r0 = (blk / ncb) << 2, c0 = (blk % ncb) << 2;
            float acc[4][4], acc2[4][4];
            zero(acc);
            zero(acc2);
            // P^T: rows t >= s only; start at the 4-aligned row r0
            mm_tn(acc, sP + r0 * ldp, ldp, r0, sG + r0 * ldv, ldv, c0, g.C - r0);
            // Kh D = sum_c Kt[s][c] gamma[c] D[c][e]
            for (int c = 0; c < g.dk; ++c) {
                const float gm = expf(sLam[(g.C - 1) * ldk + c]);
                const float4 d4 = *reinterpret_cast<const float4 *>(sD + c * ldv + c0);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float kh = sK[(r0 + i) * ldk + c] * gm;
                    acc2[i][0] += kh * d4.x; acc2[i][1] += kh * d4.y; acc2[i][2] += kh * d4.z; acc2[i][3] += kh * d4.w;
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int p = chunk * g.C + r0 + i;
                if (p < g.L) {
                    const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
                    store4(dv + tok_offset(g, b, t, h, g.dv) + c0,
                           make_float4(acc[i][0] + acc2[i][0], acc[i][1] + acc2[i][1],
                                       acc[i][2] + acc2[i][2], acc[i][3] + acc2[i][3]));
                }
            }
        }
    }

    // dq, dk for the same (row, channel) block; x = q*dq - k*dk goes to sX for the gate gradient
    {
        const int nrb = g.C >> 2, ncb = g.dk >> 2;
        for (int blk = threadIdx.x; blk < nrb * ncb; blk += kThreads) {
            const int r0 = (blk / ncb) << 2, c0 = (blk % ncb) << 2;
            float aq[4][4], ak[4][4], ak2[4][4];
            zero(aq); zero(ak); zero(ak2);
            mm_nn(aq, sdP, ldp, r0, sK, ldk, c0, r0 + 4);                          // dP Kt
            mm_nt(aq, sG, ldv, r0, sS, ldv, c0, 1, g.dv);                          // dO S^T
            mm_tn(ak, sdP + r0 * ldp, ldp, r0, sQ + r0 * ldk, ldk, c0, g.C - r0);  // dP^T Qt
            mm_nt(ak2, sV, ldv, r0, sD, ldv, c0, 1, g.dv);                         // V D^T
            const float4 last = *reinterpret_cast<const float4 *>(sLam + (g.C - 1) * ldk + c0);
            const float lc[4] = {last.x, last.y, last.z, last.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int p = chunk * g.C + r0 + i;
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (p < g.L) {
                    const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
                    const size_t off = tok_offset(g, b, t, h, g.dk) + c0;
                    const float4 lam = *reinterpret_cast<const float4 *>(sLam + (r0 + i) * ldk + c0);
                    const float lv[4] = {lam.x, lam.y, lam.z, lam.w};
                    float dqv[4], dkv[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        dqv[j] = aq[i][j] * expf(lv[j]);
                        dkv[j] = ak[i][j] * expf(-lv[j]) + ak2[i][j] * expf(lc[j] - lv[j]);
                    }
                    store4(dq + off, make_float4(dqv[0], dqv[1], dqv[2], dqv[3]));
                    store4(dk + off, make_float4(dkv[0], dkv[1], dkv[2], dkv[3]));
                    const float4 qq = load4(q + off), kk = load4(k + off);
                    x = make_float4(qq.x * dqv[0] - kk.x * dkv[0], qq.y * dqv[1] - kk.y * dkv[1],
                                    qq.z * dqv[2] - kk.z * dkv[2], qq.w * dqv[3] - kk.w * dkv[3]);
                }
                *reinterpret_cast<float4 *>(sX + (r0 + i) * ldk + c0) = x;
            }
        }
    }
    __syncthreads();
    // gate gradient: suffix sum of x down the chunk plus what later chunks carry in
    for (int c = threadIdx.x; c < g.dk; c += kThreads) {
        float run = carry[((size_t)bh * g.N + chunk) * g.dk + c];
        for (int j = g.C - 1; j >= 0; --j) {
            const int p = chunk * g.C + j;
            if (p >= g.L) continue;
            run += sX[j * ldk + c];
            const int t = scan_token(p, g.dir, g.gh, g.gw, g.L);
            dgate[tok_offset(g, b, t, h, g.dk) + c] = run;
        }
    }
}

size_t smem_state(const Geom &g, bool bwd)
{
    const size_t ldk = g.dk + 4, ldv = g.dv + 4;
    return sizeof(float) * (size_t)g.C * (ldk + ldv) * (bwd ? 2 : 1);
}
size_t smem_out(const Geom &g)
{
    const size_t ldk = g.dk + 4, ldv = g.dv + 4, ldp = g.C + 4;
    size_t n = (size_t)g.C * (3 * ldk + ldv) + (size_t)g.dk * ldv;
    if (g.C > g.dk) n += (size_t)g.C * ldp;
    return sizeof(float) * n;
}
size_t smem_bwd(const Geom &g)
{
    const size_t ldk = g.dk + 4, ldv = g.dv + 4, ldp = g.C + 4;
    return sizeof(float) * ((size_t)g.C * (4 * ldk + 2 * ldv + 2 * ldp) + 2 * (size_t)g.dk * ldv);
}
constexpr size_t kMaxSmem = 227 * 1024;

template <typename K>
dig_status set_smem(K kernel, size_t bytes)
{
    if (bytes > kMaxSmem) return DIG_ERR_UNSUPPORTED;
    return ensure_dynamic_smem(reinterpret_cast<const void *>(kernel), bytes);
}

template <typename T, typename TO>
dig_status fwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, false);
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = fma_chunk_state<T, false>;
    if ((st = set_smem(k1, smem_state(g, false))) != DIG_OK) return st;
    { KernelTimer t(KID_FMA_STATE, a.stream);
    k1<<<grid, kThreads, smem_state(g, false), a.stream>>>(
        (const T *)a.q, (const T *)a.k, (const T *)a.v, a.gate, nullptr, w.states, w.gamma, nullptr, g); }
    if ((st = launch_state_scan_fwd(w, g, a.stream, a.sio)) != DIG_OK) return st;
    auto k3 = fma_chunk_out<T, TO>;
    if ((st = set_smem(k3, smem_out(g))) != DIG_OK) return st;
    KernelTimer t(KID_FMA_OUT, a.stream);
    k3<<<grid, kThreads, smem_out(g), a.stream>>>((const T *)a.q, (const T *)a.k, (const T *)a.v,
                                                  a.gate, w.states, (TO *)a.out, g);
    return cuda_ok(cudaGetLastError());
}

template <typename T, typename TO>
dig_status bwd_typed(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, true);
    const dim3 grid(g.N, g.B * g.H);
    dig_status st;
    auto k1 = fma_chunk_state<T, true>;
    if ((st = set_smem(k1, smem_state(g, true))) != DIG_OK) return st;
    auto k4 = fma_chunk_bwd<T, TO>;
    if ((st = set_smem(k4, smem_bwd(g))) != DIG_OK) return st;
    { KernelTimer t(KID_FMA_STATE, a.stream);
    k1<<<grid, kThreads, smem_state(g, true), a.stream>>>(
        (const T *)a.q, (const T *)a.k, (const T *)a.v, a.gate, (const T *)a.d_out, w.states, w.gamma,
        w.dstates, g); }
    if ((st = launch_state_scan_fwd(w, g, a.stream, a.sio)) != DIG_OK) return st;
    if ((st = launch_state_scan_bwd(w, g, a.stream, a.sio)) != DIG_OK) return st;
    KernelTimer t(KID_FMA_BWD, a.stream);
    k4<<<grid, kThreads, smem_bwd(g), a.stream>>>(
        (const T *)a.q, (const T *)a.k, (const T *)a.v, a.gate, (const T *)a.d_out, w.states, w.dstates,
        w.carry, (TO *)a.dq, (TO *)a.dk, (TO *)a.dv, a.dgate, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

bool fma_supports(int dk, int dv, int chunk, int dtype, bool backward)
{
    (void)dtype;
    Geom g{};
    g.dk = dk; g.dv = dv; g.C = chunk;
    if (backward) return smem_bwd(g) <= kMaxSmem && smem_state(g, true) <= kMaxSmem;
    return smem_out(g) <= kMaxSmem && smem_state(g, false) <= kMaxSmem;
}

dig_status fma_gla_fwd(const GlaArgs &a)
{
    switch (a.dtype) {
        case DIG_F32: return fwd_typed<float, float>(a);
        case DIG_BF16: return fwd_typed<__nv_bfloat16, __nv_bfloat16>(a);
        case DIG_BF16_F32OUT: return fwd_typed<__nv_bfloat16, float>(a);
    }
    return DIG_ERR_INVALID_ARG;
}

dig_status fma_gla_bwd(const GlaArgs &a)
{
    switch (a.dtype) {
        case DIG_F32: return bwd_typed<float, float>(a);
        case DIG_BF16: return bwd_typed<__nv_bfloat16, __nv_bfloat16>(a);
        case DIG_BF16_F32OUT: return bwd_typed<__nv_bfloat16, float>(a);
    }
    return DIG_ERR_INVALID_ARG;
}

}  // namespace dig
