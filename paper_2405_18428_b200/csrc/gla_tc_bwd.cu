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
// kernel and are bulk-copied (cp.async.bulk) straight into their operand tiles; q, k, v, dO and
// gate rows of the next chunk are prefetched into registers.  A seventeenth warp issues the MMAs
// and the bulk copies, so the tensor pipe runs while the other warps build operands.  Results are
// staged in shared memory and leave with coalesced 16-byte stores.
#include "tc_tiles.cuh"

namespace dig {
namespace {

using namespace tc;

constexpr int NT = 512;                      // threads that build operands and post-process accumulators
constexpr int NTA = NT + 32;                 // plus one warp that issues the MMAs and the bulk loads
constexpr int W = 16;                         // accumulator columns per thread
constexpr int kTile = T * 64 * 4;             // one 64 x 64 operand tile
constexpr int kLamBytes = T * kLamPitch * 4;

struct BwdRaw {
    uint4 q, k, v, d;
    float4 gt[2];
};

__device__ __forceinline__ void load_raw(BwdRaw &r, const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *d_out,
                                         const float *gate, const Geom &g, const Item &it)
{
    // 8 lanes cover one 128-byte bf16 row; the same lanes take the 8 gates of their columns
    const int row = threadIdx.x >> 3, col = (threadIdx.x & 7) * 8;
    const size_t off = row_offset(g, it, row) + col;
    r.q = ldg16(q + off);
    r.k = ldg16(k + off);
    r.v = ldg16(v + off);
    r.d = ldg16(d_out + off);
    const int fl = col >= 32 ? 4 : 0;         // flipped lanes hold their upper four columns first
    r.gt[0] = ldg16(gate + off + fl);
    r.gt[1] = ldg16(gate + off + 4 - fl);
}

// State entering the chunk, and the decayed state gradient leaving it in both tile orders:
// 16 KB each, written by the scan kernel exactly as the operand tiles want them.
__device__ __forceinline__ void fetch_states(char *tSk, char *tDk, char *tDm, const float *states, const float *dstates,
                                             const float *dstates_m, int id, uint64_t *bar)
{
    fence_async_smem();
    mbar_arrive_expect_tx(bar, 3u * kTile);
    bulk_g2s(tSk, states + (size_t)id * (DK * DV), kTile, bar);
    bulk_g2s(tDk, dstates + (size_t)id * (DK * DV), kTile, bar);
    bulk_g2s(tDm, dstates_m + (size_t)id * (DK * DV), kTile, bar);
}

template <typename TO>
__global__ void __launch_bounds__(NTA)
tc_chunk_bwd(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
             const float *__restrict__ gate, const bf16 *__restrict__ d_out, const float *__restrict__ states,
             const float *__restrict__ dstates, const float *__restrict__ dstates_m, const float *__restrict__ carry,
             TO *__restrict__ dq,
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
    // results are staged over tiles 0-3 once every product has completed
    constexpr int kOutPitch = 64 * (int)sizeof(TO) + 16, kOutStage = T * kOutPitch;
    static_assert(3 * kOutStage <= 4 * kTile, "output staging must fit in the four tiles it reuses");
    char *stage = base;
    float *sLamBuf = reinterpret_cast<float *>(base + 10 * kTile);          // gate table, later q*dq - k*dk and the gate gradient
    float *sLast = sLamBuf + T * kLamPitch, *sTot = sLast + 64;
    Control *ctl = reinterpret_cast<Control *>(sTot + NT);
    uint64_t *barA = &ctl->bar[0], *barB = &ctl->bar[1], *barS = &ctl->bar[2];
    constexpr uint32_t kCols = 256;
    constexpr uint32_t aP = 0, aQK = 64, aV = 128, kUpper = 16u << 16;      // upper half of a lane quarter
    setup(ctl, 4, kCols);
    const uint32_t tmem = ctl->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool issuer = warp == NT / 32;                                    // the extra warp: MMAs and bulk loads
    const int hf = lane >> 4, arow = 16 * (warp & 3) + (lane & 15), c0 = W * ((warp >> 2) & 3);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;

    const int total = g.B * g.H * g.N;
    BwdRaw raw;
    int id = blockIdx.x;
    Item it = item_of(g, id, total);
    // q, k, v, dO and the gates are inputs of the whole call: their loads need not wait for the scan
    // kernel that is still finishing; the states and carries it writes do
    if (id < total && !issuer) load_raw(raw, q, k, v, d_out, gate, g, it);
    pdl_wait();
    pdl_launch_dependents();          // only once this kernel's own predecessor has completed
    if (id < total && issuer && lane == 0) fetch_states(tSk, tDk, tDm, states, dstates, dstates_m, id, barS);
    uint32_t parity = 0;
    bool ok = true;
    for (; id < total; id += gridDim.x) {
        float *sLam = sLamBuf;
        const int next = id + gridDim.x;
        const Item nit = item_of(g, next, total);
        const int row = threadIdx.x >> 3, j = threadIdx.x & 7, col = j * 8;
        const bool flip = j >= 4;
        const bool keep = it.chunk * T + row < g.L;
        float carry_in = 0.f;
        if (!issuer) {
            carry_in = __ldg(carry + (size_t)id * DK + (threadIdx.x & 63));
            sync_group(NT);              // the previous chunk's results have left the staging area
            float x[8];
            unpack8(raw.v, x, keep, flip);
            st_k8<T, false>(tVk, row, col, x, flip);
            unpack8(raw.d, x, keep, flip);
            st_k8<T, false>(tGk, row, col, x, flip);
            st_m8<T, false>(tGm, row, col, x, flip);
            fence_async_smem();
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (issuer) {
            if (lane == 0) {
                // products of operands that need no gate: they run while the other warps build Qt and Kt
                ok = mbar_wait(barS, parity, status);      // S, Dg (both tile orders) have landed
                tc_fence_after_sync();
                issue<64, 64, false, false, T, T>(tmem + aQK, kdesc<T>(tGk), kdesc<T>(tSk), false);             // dO S^T
                issue<64, 64, false, false, T, T>(tmem + aQK + kUpper, kdesc<T>(tVk), kdesc<T>(tDk), false);    // V Dg^T
                issue<64, 64, false, false, T, T>(tmem + aP + kUpper, kdesc<T>(tGk), kdesc<T>(tVk), false);     // dO V^T
            }
        } else {
            {
                const float sc = keep ? kLog2e : 0.f;
                float *dst = sLam + row * kLamPitch + col;
                const int fl = flip ? 4 : 0;
                *reinterpret_cast<float4 *>(dst + fl) = make_float4(raw.gt[0].x * sc, raw.gt[0].y * sc, raw.gt[0].z * sc, raw.gt[0].w * sc);
                *reinterpret_cast<float4 *>(dst + 4 - fl) = make_float4(raw.gt[1].x * sc, raw.gt[1].y * sc, raw.gt[1].z * sc, raw.gt[1].w * sc);
            }
            sync_group(NT);
            gate_prefix<NT, 1, true>(sLam, sLast, sTot);
            float lam[8], x[8];
            read_lam8(sLam, row, col, lam, flip);
            unpack8(raw.q, x, keep, flip);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = to_tf32(x[e] * ex2(lam[e]));
            st_k8<T, false>(tQk, row, col, x, flip);
            st_m8<T, false>(tQm, row, col, x, flip);
            unpack8(raw.k, x, keep, flip);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = to_tf32(x[e] * ex2(-lam[e]));
            st_k8<T, false>(tKk, row, col, x, flip);
            st_m8<T, false>(tKm, row, col, x, flip);
            fence_async_smem();
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (issuer) {
            if (lane == 0) {
                tc_fence_after_sync();
                issue<64, 64, false, false, T, T>(tmem + aP, kdesc<T>(tQk), kdesc<T>(tKk), false);              // Qt Kt^T
                mma_commit(barA);
                issue<64, 64, false, true, T, T>(tmem + aV, kdesc<T>(tKk), mdesc<T>(tDm), false);               // Kt Dg
            }
        } else {
            ok = mbar_wait(barA, parity, status);
            if (ok) {
                tc_fence_after_sync();
                float p[W];
                tmem_ld(tmem + lane_base + aP + (uint32_t)c0, p);       // lanes 0-15: scores, lanes 16-31: dO V^T
#pragma unroll
                for (int jj = 0; jj < W; ++jj)
                    p[jj] = c0 + jj > arow ? 0.f : to_tf32(p[jj]);       // keep s <= t; the diagonal has weight 1
                if (hf == 0) {
#pragma unroll
                    for (int jj = 0; jj < W / 4; ++jj)
                        st_m4<T, false>(tPm, arow, c0 + 4 * jj, make_float4(p[4 * jj], p[4 * jj + 1], p[4 * jj + 2], p[4 * jj + 3]));
                } else {
#pragma unroll
                    for (int jj = 0; jj < W / 4; ++jj) {
                        const float4 v4 = make_float4(p[4 * jj], p[4 * jj + 1], p[4 * jj + 2], p[4 * jj + 3]);
                        st_k4<T, false>(tdPk, arow, c0 + 4 * jj, v4);
                        st_m4<T, false>(tdPm, arow, c0 + 4 * jj, v4);
                    }
                }
            }
            fence_async_smem();
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (issuer) {
            if (lane == 0) {
                tc_fence_after_sync();
                issue<64, 64, false, true, T, T>(tmem + aQK, kdesc<T>(tdPk), mdesc<T>(tKm), true);              // + dP Kt
                issue<64, 64, true, true, T, T>(tmem + aQK + kUpper, mdesc<T>(tdPm), mdesc<T>(tQm), true);      // + dP^T Qt
                issue<64, 64, true, true, T, T>(tmem + aV, mdesc<T>(tPm), mdesc<T>(tGm), true);                 // + P^T dO
                mma_commit(barB);
                // once everything has completed the state tiles are free for the next chunk
                if (mbar_wait(barB, parity, status) && next < total) fetch_states(tSk, tDk, tDm, states, dstates, dstates_m, next, barS);
            }
        } else {
            // the tensor pipe is busy for a while: a good moment to start the next chunk's loads
            if (next < total) load_raw(raw, q, k, v, d_out, gate, g, nit);
            ok = mbar_wait(barB, parity, status);
            if (ok) {
                tc_fence_after_sync();
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
                store16(reinterpret_cast<TO *>(stage + hf * kOutStage + arow * kOutPitch) + c0, a);      // dq | dk
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
                if (hf == 0) store16(reinterpret_cast<TO *>(stage + 2 * kOutStage + arow * kOutPitch) + c0, a);
            }
            tc_fence_before_sync();
            sync_group(NT);
            {
                // gate gradient: suffix sums of x down the chunk plus what later chunks carry in, in place
                constexpr int R = T / (NT / 64);        // rows per thread
                const int c = threadIdx.x & 63, seg = threadIdx.x >> 6;
                float s[R];
#pragma unroll
                for (int jj = 0; jj < R; ++jj) s[jj] = sLam[(R * seg + jj) * kLamPitch + c];
#pragma unroll
                for (int jj = R - 2; jj >= 0; --jj) s[jj] += s[jj + 1];
                sTot[seg * 64 + c] = s[0];
                sync_group(NT);
                float add = carry_in;
#pragma unroll
                for (int sg = 1; sg < NT / 64; ++sg)
                    if (sg > seg) add += sTot[sg * 64 + c];
#pragma unroll
                for (int jj = 0; jj < R; ++jj) sLam[(R * seg + jj) * kLamPitch + c] = s[jj] + add;
            }
            sync_group(NT);
            if (ok) {
                // coalesced stores of the staged results: 16 bytes per thread, 8 or 16 threads per token row
                constexpr int PER_ROW = 64 * (int)sizeof(TO) / 16;
#pragma unroll
                for (int i = 0; i < PER_ROW / 8; ++i) {
                    const int u = threadIdx.x + NT * i, r = u / PER_ROW, piece = u % PER_ROW;
                    const int tr = item_token(g, it, r);
                    if (tr >= 0) {
                        const size_t off = tok_offset(g, it.b, tr, it.h, 64) * sizeof(TO) + piece * 16;
                        const char *src = stage + r * kOutPitch + piece * 16;
                        *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(dq) + off) = *reinterpret_cast<const uint4 *>(src);
                        *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(dk) + off) = *reinterpret_cast<const uint4 *>(src + kOutStage);
                        *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(dv) + off) = *reinterpret_cast<const uint4 *>(src + 2 * kOutStage);
                    }
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int u = threadIdx.x + NT * i, r = u >> 4, c4 = (u & 15) * 4;
                    const int tr = item_token(g, it, r);
                    if (tr >= 0)
                        *reinterpret_cast<float4 *>(dgate + tok_offset(g, it.b, tr, it.h, DK) + c4) =
                            *reinterpret_cast<const float4 *>(sLam + r * kLamPitch + c4);
                }
            }
        }
        parity ^= 1;
        it = nit;
    }
    if (!ok) {      // a wait gave up: let bulk copies still in flight land before the CTA's memory goes away
        mbar_wait(barS, parity, status);
    }
    teardown(ctl, kCols);
}

constexpr size_t bwd_smem()
{
    return 1024 + 10 * (size_t)kTile + kLamBytes + sizeof(float) * (64 + NT) + sizeof(Control);
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
    launch_pdl(kern, dim3(grid), dim3(NTA), smem, a.stream, (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate,
               (const bf16 *)a.d_out, (const float *)w.states, (const float *)w.dstates, (const float *)w.dstates_m,
               (const float *)w.carry, (TO *)a.dq, (TO *)a.dk, (TO *)a.dv, a.dgate, status, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

dig_status launch_tc_bwd(const GlaArgs &a, const Workspace &w, int sm_count, int *status)
{
    return a.dtype == DIG_BF16 ? launch_typed<bf16>(a, w, sm_count, status) : launch_typed<float>(a, w, sm_count, status);
}

}  // namespace dig
