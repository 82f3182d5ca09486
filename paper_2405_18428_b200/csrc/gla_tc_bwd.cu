// Tensor-core gradient kernel of chunkwise gated linear attention (reverse mode of Eq. attn_gla,
// evaluated chunk by chunk as in Section 3.5).  Per chunk, with Lam the in-chunk cumulative gate,
// Qt = q*exp(Lam), Kt = k*exp(-Lam), S the state entering the chunk and Dg = diag(gamma) dL/dS_out:
//   P  = tril(Qt Kt^T),  dP = tril(dO V^T)
//   dq = (dP Kt + dO S^T) * exp(Lam)
//   dk = (dP^T Qt + V Dg^T) * exp(-Lam)
//   dv = P^T dO + Kt Dg
//   dgate_j = carry + sum_{r >= j in chunk} (q*dq - k*dk)_r
//
// One persistent CTA of 512 threads per SM walks over the chunks.  Every product is a 64 x 64 x 64
// tcgen05.mma (kind::tf32) sequence; a 64-row accumulator only fills lanes 0-15 of each 32-lane
// quarter of tensor memory, so two accumulators that are post-processed alike share their columns:
// P / dP and dq / dk sit in lanes 0-15 / 16-31 of the same columns and every thread of a warp has
// one accumulator row to work on.  S and Dg arrive tf32-rounded and in tile order from the scan
// kernel and are bulk-copied straight into their operand tiles; gate rows are bulk-copied into a
// double-buffered table; q, k, v, dO rows of the next chunk are prefetched into registers.
#include "tc_tiles.cuh"

namespace dig {
namespace {

using namespace tc;

constexpr int NT = 512;
constexpr int W = 16;                         // accumulator columns per thread
constexpr int kTile = T * 64 * 4;             // one 64 x 64 operand tile
constexpr int kLamBytes = T * kLamPitch * 4;

struct BwdRaw {
    uint4 q, k, v, d;
};

__device__ __forceinline__ void load_raw(BwdRaw &r, const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *d_out,
                                         const Geom &g, const Item &it)
{
    const int row = threadIdx.x >> 3, col = (threadIdx.x & 7) * 8;
    const int tok = item_token(g, it, row);
    r.q = ld_row8(q, g, it.b, tok, it.h, DK, col);
    r.k = ld_row8(k, g, it.b, tok, it.h, DK, col);
    r.v = ld_row8(v, g, it.b, tok, it.h, DV, col);
    r.d = ld_row8(d_out, g, it.b, tok, it.h, DV, col);
}

// State entering the chunk and decayed state gradient leaving it: 16 KB each, already in tile order.
__device__ __forceinline__ void fetch_states(char *tSk, char *tDk, const float *states, const float *dstates, int id,
                                             uint64_t *bar)
{
    fence_async_smem();
    mbar_arrive_expect_tx(bar, 2u * kTile);
    bulk_g2s(tSk, states + (size_t)id * (DK * DV), kTile, bar);
    bulk_g2s(tDk, dstates + (size_t)id * (DK * DV), kTile, bar);
}

template <typename TO>
__global__ void __launch_bounds__(NT)
tc_chunk_bwd(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
             const float *__restrict__ gate, const bf16 *__restrict__ d_out, const float *__restrict__ states,
             const float *__restrict__ dstates, const float *__restrict__ carry, TO *__restrict__ dq,
             TO *__restrict__ dk, TO *__restrict__ dv, float *__restrict__ dgate, int *status, Geom g)
{
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    // K-format tiles
    char *tQk = base + 0 * kTile, *tKk = base + 1 * kTile, *tVk = base + 2 * kTile, *tGk = base + 3 * kTile;
    char *tSk = base + 4 * kTile, *tDk = base + 5 * kTile;
    // M-format tiles
    char *tQm = base + 6 * kTile, *tKm = base + 7 * kTile, *tGm = base + 8 * kTile, *tDm = base + 9 * kTile;
    // written after the first group of products has completed, over tiles that group has finished with
    char *tPm = tQk, *tdPk = tVk, *tdPm = tSk;
    float *sLamBuf = reinterpret_cast<float *>(base + 10 * kTile);          // two gate tables
    float *sLast = sLamBuf + 2 * T * kLamPitch, *sTot = sLast + 64;
    Control *ctl = reinterpret_cast<Control *>(sTot + NT);
    uint64_t *barA = &ctl->bar[0], *barB = &ctl->bar[1], *barG = &ctl->bar[2], *barS = &ctl->bar[3];
    constexpr uint32_t kCols = 256;
    constexpr uint32_t aP = 0, aQK = 64, aV = 128, kUpper = 16u << 16;      // upper half of a lane quarter
    setup(ctl, 4, kCols, 2, 2);
    const uint32_t tmem = ctl->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int hf = lane >> 4, arow = 16 * (warp & 3) + (lane & 15), c0 = W * (warp >> 2);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;

    const int total = g.B * g.H * g.N;
    BwdRaw raw;
    int id = blockIdx.x;
    if (id < total) {
        const Item it = item_of(g, id, total);
        load_raw(raw, q, k, v, d_out, g, it);
        if (warp == 4 || warp == 5) fetch_gate_rows(sLamBuf, gate, g, it, warp - 4, barG, lane);
        if (threadIdx.x == 0) fetch_states(tSk, tDk, states, dstates, id, barS);
    }
    uint32_t parity = 0;
    bool ok = true;
    for (; id < total; id += gridDim.x) {
        float *sLam = sLamBuf + parity * (T * kLamPitch);
        const Item it = item_of(g, id, total);
        const int next = id + gridDim.x;
        const Item nit = item_of(g, next, total);
        ok = mbar_wait(barG, parity, status);
        if (!__syncthreads_and(ok)) break;
        gate_prefix<NT, 1>(sLam, sLast, sTot, kLog2e);
        {
            const int row = threadIdx.x >> 3, j = threadIdx.x & 7, col = j * 8;
            const bool flip = j >= 4;
            const bool keep = it.chunk * T + row < g.L;
            float lam[8], x[8];
            read_lam8(sLam, row, col, lam);
            unpack8(raw.q, x, keep);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = to_tf32(x[e] * ex2(lam[e]));
            st_k8<T, false>(tQk, row, col, x, flip);
            st_m8<T, false>(tQm, row, col, x, flip);
            unpack8(raw.k, x, keep);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = to_tf32(x[e] * ex2(-lam[e]));
            st_k8<T, false>(tKk, row, col, x, flip);
            st_m8<T, false>(tKm, row, col, x, flip);
            unpack8(raw.v, x, keep);
            st_k8<T, false>(tVk, row, col, x, flip);
            unpack8(raw.d, x, keep);
            st_k8<T, false>(tGk, row, col, x, flip);
            st_m8<T, false>(tGm, row, col, x, flip);
            // Dg also in M-format (same values, other piece order inside the row)
            ok = mbar_wait(barS, parity, status);
            if (ok) {
                const char *src = tDk + (j >> 2) * (T * 128) + row * 128;
                const int c = 2 * (j & 3), s = row & 7;
                const float4 lo = *reinterpret_cast<const float4 *>(src + ((c ^ s) << 4));
                const float4 hi = *reinterpret_cast<const float4 *>(src + (((c + 1) ^ s) << 4));
                const float y[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
                st_m8<T, false>(tDm, row, col, y, flip);
            }
        }
        fence_async_smem();
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (threadIdx.x == 0) {
            tc_fence_after_sync();
            issue<64, 64, false, false, T, T>(tmem + aQK, kdesc<T>(tGk), kdesc<T>(tSk), false);             // dO S^T
            issue<64, 64, false, false, T, T>(tmem + aQK + kUpper, kdesc<T>(tVk), kdesc<T>(tDk), false);    // V Dg^T
            issue<64, 64, false, false, T, T>(tmem + aP, kdesc<T>(tQk), kdesc<T>(tKk), false);              // Qt Kt^T
            issue<64, 64, false, false, T, T>(tmem + aP + kUpper, kdesc<T>(tGk), kdesc<T>(tVk), false);     // dO V^T
            mma_commit(barA);
            issue<64, 64, false, true, T, T>(tmem + aV, kdesc<T>(tKk), mdesc<T>(tDm), false);               // Kt Dg
        }
        if (next < total) {
            if (warp == 4 || warp == 5)
                fetch_gate_rows(sLamBuf + (parity ^ 1) * (T * kLamPitch), gate, g, nit, warp - 4, barG, lane);
            load_raw(raw, q, k, v, d_out, g, nit);
        }
        ok = mbar_wait(barA, parity, status);
        if (ok) {
            tc_fence_after_sync();
            float p[W];
            tmem_ld(tmem + lane_base + aP + (uint32_t)c0, p);       // lanes 0-15: scores, lanes 16-31: dO V^T
#pragma unroll
            for (int jj = 0; jj < W; ++jj)
                if (c0 + jj > arow) p[jj] = 0.f;                     // keep s <= t; the diagonal has weight 1
            if (hf == 0) {
#pragma unroll
                for (int jj = 0; jj < W / 4; ++jj)
                    st_m4<T>(tPm, arow, c0 + 4 * jj, make_float4(p[4 * jj], p[4 * jj + 1], p[4 * jj + 2], p[4 * jj + 3]));
            } else {
#pragma unroll
                for (int jj = 0; jj < W / 4; ++jj) {
                    const float4 v4 = make_float4(p[4 * jj], p[4 * jj + 1], p[4 * jj + 2], p[4 * jj + 3]);
                    st_k4<T>(tdPk, arow, c0 + 4 * jj, v4);
                    st_m4<T>(tdPm, arow, c0 + 4 * jj, v4);
                }
            }
        }
        fence_async_smem();
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (threadIdx.x == 0) {
            tc_fence_after_sync();
            issue<64, 64, false, true, T, T>(tmem + aQK, kdesc<T>(tdPk), mdesc<T>(tKm), true);              // + dP Kt
            issue<64, 64, true, true, T, T>(tmem + aQK + kUpper, mdesc<T>(tdPm), mdesc<T>(tQm), true);      // + dP^T Qt
            issue<64, 64, true, true, T, T>(tmem + aV, mdesc<T>(tPm), mdesc<T>(tGm), true);                 // + P^T dO
            mma_commit(barB);
        }
        ok = mbar_wait(barB, parity, status);
        if (ok) {
            tc_fence_after_sync();
            if (threadIdx.x == 0 && next < total) fetch_states(tSk, tDk, states, dstates, next, barS);     // tiles are free again
            const int tok = item_token(g, it, arow);
            float a[W], lam[W], x[W];
#pragma unroll
            for (int jj = 0; jj < W / 4; ++jj) {
                const float4 l4 = *reinterpret_cast<const float4 *>(sLam + arow * kLamPitch + c0 + 4 * jj);
                lam[4 * jj] = l4.x; lam[4 * jj + 1] = l4.y; lam[4 * jj + 2] = l4.z; lam[4 * jj + 3] = l4.w;
            }
            tmem_ld(tmem + lane_base + aQK + (uint32_t)c0, a);      // lanes 0-15: dq part, lanes 16-31: dk part
            {
                // q*dq = Qt*(dq accumulator), k*dk = Kt*(dk accumulator): the decay factors cancel
                float t8[8];
                ld_m8<T>(hf == 0 ? tQm : tKm, arow, c0, t8);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] = t8[e] * a[e];
                ld_m8<T>(hf == 0 ? tQm : tKm, arow, c0 + 8, t8);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[8 + e] = t8[e] * a[8 + e];
            }
#pragma unroll
            for (int jj = 0; jj < W; ++jj) a[jj] *= ex2(hf == 0 ? lam[jj] : -lam[jj]);
            if (tok >= 0) store16((hf == 0 ? dq : dk) + tok_offset(g, it.b, tok, it.h, DK) + c0, a);
            __syncwarp();            // both halves have read their gates before the table is overwritten
#pragma unroll
            for (int jj = 0; jj < W; ++jj) {
                const float other = __shfl_xor_sync(0xffffffffu, x[jj], 16);
                x[jj] -= other;                                      // lanes 0-15: q*dq - k*dk
            }
            if (hf == 0) {
#pragma unroll
                for (int jj = 0; jj < W / 4; ++jj)
                    *reinterpret_cast<float4 *>(sLam + arow * kLamPitch + c0 + 4 * jj) =
                        make_float4(x[4 * jj], x[4 * jj + 1], x[4 * jj + 2], x[4 * jj + 3]);
            }
            tmem_ld(tmem + lane_base + aV + (uint32_t)c0, a);       // warp-wide instruction; only lanes 0-15 hold dv rows
            if (hf == 0 && tok >= 0) store16(dv + tok_offset(g, it.b, tok, it.h, DV) + c0, a);
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        tc_fence_after_sync();
        {
            // gate gradient: suffix sums of x down the chunk plus what later chunks carry in
            constexpr int R = T / (NT / 64);        // rows per thread
            const int c = threadIdx.x & 63, seg = threadIdx.x >> 6;
            float s[R];
#pragma unroll
            for (int jj = 0; jj < R; ++jj) s[jj] = sLam[(R * seg + jj) * kLamPitch + c];
#pragma unroll
            for (int jj = R - 2; jj >= 0; --jj) s[jj] += s[jj + 1];
            sTot[seg * 64 + c] = s[0];
            __syncthreads();
            float add = __ldg(carry + (size_t)id * DK + c);
#pragma unroll
            for (int sg = 1; sg < NT / 64; ++sg)
                if (sg > seg) add += sTot[sg * 64 + c];
#pragma unroll
            for (int jj = 0; jj < R; ++jj) {
                const int tj = item_token(g, it, R * seg + jj);
                if (tj >= 0) dgate[tok_offset(g, it.b, tj, it.h, DK) + c] = s[jj] + add;
            }
        }
        parity ^= 1;
        __syncthreads();
    }
    if (!ok) {      // a wait gave up: let bulk copies still in flight land before the CTA's memory goes away
        mbar_wait(barG, parity, status);
        mbar_wait(barS, parity, status);
    }
    teardown(ctl, kCols);
}

constexpr size_t bwd_smem()
{
    return 1024 + 10 * (size_t)kTile + 2 * kLamBytes + sizeof(float) * (64 + NT) + sizeof(Control);
}

template <typename TO>
dig_status launch_typed(const GlaArgs &a, const Workspace &w, int sm_count, int *status)
{
    const Geom &g = a.g;
    const int total = g.B * g.H * g.N;
    auto kern = tc_chunk_bwd<TO>;
    constexpr size_t smem = bwd_smem();
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DIG_ERR_CUDA;
    const int grid = total < sm_count ? total : sm_count;
    KernelTimer t(KID_TC_BWD, a.stream);
    kern<<<grid, NT, smem, a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate,
                                       (const bf16 *)a.d_out, w.states, w.dstates, w.carry, (TO *)a.dq, (TO *)a.dk,
                                       (TO *)a.dv, a.dgate, status, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

dig_status launch_tc_bwd(const GlaArgs &a, const Workspace &w, int sm_count, int *status)
{
    return a.dtype == DIG_BF16 ? launch_typed<bf16>(a, w, sm_count, status) : launch_typed<float>(a, w, sm_count, status);
}

}  // namespace dig
