// Tensor-core output kernel of chunkwise gated linear attention (Eq. attn_gla, Section 3.5):
//   out = tril(Qt Kt^T) V + Qt S,   Qt = q*exp(Lam), Kt = k*exp(-Lam),
// S the state entering the chunk (read as S^T, [d_v][d_k], from the workspace).
//
// A persistent CTA of 512 threads works on two chunks at a time, stacked along the M dimension
// of tcgen05.mma (rows 0-63 chunk a, rows 64-127 chunk b).  The B operands of the two chunks are
// concatenated along N, so every product is 8 instructions of M = N = 128 for both chunks:
//   scores  [Qa;Qb] [Ka;Kb]^T      -> wanted blocks (a, cols 0-63), (b, cols 64-127)
//   inter   [Qa;Qb] [Sa^T;Sb^T]^T  -> same blocks of the output accumulator
//   intra   [Pa;Pb] [Va | Vb]      -> accumulated on top
// The other blocks of the accumulators hold cross terms that are never read.  While a pair is in
// the tensor pipe the next pair's q, k, v and gate rows are already being loaded into registers, and
// its incoming states arrive by bulk asynchronous copies (cp.async.bulk) in their operand tile.  A
// seventeenth warp issues the MMAs and the bulk copies; results leave through a staging area with
// coalesced 16-byte stores.
#include "tc_tiles.cuh"

namespace dig {
namespace {

using namespace tc;

constexpr int NT = 512;                       // threads that build operands and post-process accumulators
constexpr int NTA = NT + 32;                  // plus one warp that issues the MMAs and the bulk loads
constexpr int W = 16;                          // accumulator columns per thread
constexpr int kTileK = 128 * 64 * 4;           // 128 rows x 64 columns, K-format
constexpr int kTileM = T * 128 * 4;            // 64 rows x 128 columns, M-format

struct OutRaw {
    uint4 q[2], k[2], v[2];
    float4 g0[2], g1[2];
};

// 8 lanes cover one 128-byte bf16 row; the same lanes take the 8 gates of their columns.
__device__ __forceinline__ void load_raw(OutRaw &r, const bf16 *q, const bf16 *k, const bf16 *v, const float *gate,
                                         const Geom &g, const Item (&it)[2])
{
    const int row = threadIdx.x >> 3, col = (threadIdx.x & 7) * 8;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const size_t off = row_offset(g, it[half], row) + col;
        r.q[half] = ldg16(q + off);
        r.k[half] = ldg16(k + off);
        r.v[half] = ldg16(v + off);
        const int fl = col >= 32 ? 4 : 0;     // flipped lanes hold their upper four columns first
        r.g0[half] = ldg16(gate + off + fl);
        r.g1[half] = ldg16(gate + off + 4 - fl);
    }
}

// The two chunks' incoming states (already tf32-rounded and in tile order in the workspace) go
// straight into the stacked S^T tile: per chunk one 8 KB bulk copy per column block.
__device__ __forceinline__ void fetch_states(char *tS, const float *states, int pair, int total, uint64_t *bar)
{
    fence_async_smem();
    const uint32_t n = (2 * pair + 1 < total) ? 2u : 1u;
    mbar_arrive_expect_tx(bar, n * (uint32_t)(DK * DV * 4));
    for (uint32_t half = 0; half < n; ++half) {
        const char *src = reinterpret_cast<const char *>(states + (size_t)(2 * pair + half) * (DK * DV));
        bulk_g2s(tS + half * (T * 128), src, T * 128, bar);
        bulk_g2s(tS + 128 * 128 + half * (T * 128), src + T * 128, T * 128, bar);
    }
}

template <typename TO>
__global__ void __launch_bounds__(NTA)
tc_out_pair(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
            const float *__restrict__ gate, const float *__restrict__ states, TO *__restrict__ out,
            int *status, Geom g)
{
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    char *tQ = base, *tK = base + kTileK, *tS = base + 2 * kTileK, *tP = base + 3 * kTileK;    // K-format, 128 rows
    char *tV = base + 4 * kTileK;                                                              // M-format, 64 x 128
    float *sLam = reinterpret_cast<float *>(tV + kTileM);
    float *sLast = sLam + 2 * T * kLamPitch, *sTot = sLast + 128;
    Control *ctl = reinterpret_cast<Control *>(sTot + NT);
    // results are staged over the score tile's operands (Q and K tiles) once every product has completed
    constexpr int kOutPitch = 64 * (int)sizeof(TO) + 16;
    static_assert(128 * kOutPitch <= 2 * kTileK, "output staging must fit in the tiles it reuses");
    char *stage = tQ;
    constexpr uint32_t kCols = 256;
    constexpr uint32_t aP = 0, aO = 128;
    uint64_t *barP = &ctl->bar[0], *barO = &ctl->bar[1], *barS = &ctl->bar[2];
    setup(ctl, 3, kCols);
    const uint32_t tmem = ctl->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool issuer = warp == NT / 32;                      // the extra warp: MMAs and bulk loads
    const int R = 32 * (warp & 3) + lane, half_r = R >> 6, r = R & 63, c0 = W * ((warp >> 2) & 3);
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;

    const int total = g.B * g.H * g.N, npairs = (total + 1) / 2;
    OutRaw raw;
    int pair = blockIdx.x;
    if (pair < npairs) {
        const Item it[2] = {item_of(g, 2 * pair, total), item_of(g, 2 * pair + 1, total)};
        // q, k, v and the gates are inputs of the whole call: their loads need not wait for the scan
        // kernel that is still finishing; the states it writes do
        if (!issuer) load_raw(raw, q, k, v, gate, g, it);
        pdl_wait();
        if (issuer && lane == 0) fetch_states(tS, states, pair, total, barS);
    } else {
        pdl_wait();
    }
    pdl_launch_dependents();          // only once this kernel's own predecessor has completed
    uint32_t parity = 0;
    bool ok = true;
    Item cur[2] = {item_of(g, 2 * pair, total), item_of(g, 2 * pair + 1, total)};
    for (; pair < npairs; pair += gridDim.x) {
        const int next = pair + gridDim.x;
        const Item nit[2] = {item_of(g, 2 * next, total), item_of(g, 2 * next + 1, total)};
        const int row = threadIdx.x >> 3, j = threadIdx.x & 7, col = j * 8;
        const bool flip = j >= 4;
        if (!issuer) {
            sync_group(NT);          // the previous pair's results have left the staging area
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const float sc = (cur[half].valid && cur[half].chunk * T + row < g.L) ? kLog2e : 0.f;
                float *dst = sLam + (64 * half + row) * kLamPitch + col;
                const int fl = flip ? 4 : 0;
                *reinterpret_cast<float4 *>(dst + fl) =
                    make_float4(raw.g0[half].x * sc, raw.g0[half].y * sc, raw.g0[half].z * sc, raw.g0[half].w * sc);
                *reinterpret_cast<float4 *>(dst + 4 - fl) =
                    make_float4(raw.g1[half].x * sc, raw.g1[half].y * sc, raw.g1[half].z * sc, raw.g1[half].w * sc);
            }
            sync_group(NT);
            gate_prefix<NT, 2, true>(sLam, sLast, sTot);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const bool keep = cur[half].valid && cur[half].chunk * T + row < g.L;
                float lam[8], x[8];
                read_lam8(sLam, 64 * half + row, col, lam, flip);
                unpack8(raw.q[half], x, keep, flip);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] *= ex2(lam[e]);
                st_k8<128>(tQ, 64 * half + row, col, x, flip);
                unpack8(raw.k[half], x, keep, flip);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] *= ex2(-lam[e]);
                st_k8<128>(tK, 64 * half + row, col, x, flip);
                unpack8(raw.v[half], x, keep, flip);
                st_m8<T, false>(tV, row, 64 * half + col, x, flip);
            }
            fence_async_smem();
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (issuer) {
            if (lane == 0) {
                ok = mbar_wait(barS, parity, status);
                tc_fence_after_sync();
                issue<128, 128, false, false, 128, 128>(tmem + aP, kdesc<128>(tQ), kdesc<128>(tK), false);     // scores
                mma_commit(barP);
                issue<128, 128, false, false, 128, 128>(tmem + aO, kdesc<128>(tQ), kdesc<128>(tS), false);     // Qt S
            }
        } else {
            ok = mbar_wait(barP, parity, status);
            if (ok) {
                tc_fence_after_sync();
                float p[W];
                tmem_ld(tmem + lane_base + aP + (uint32_t)(64 * half_r + c0), p);
#pragma unroll
                for (int jj = 0; jj < W; ++jj)
                    if (c0 + jj > r) p[jj] = 0.f;                   // keep s <= t; the diagonal has weight 1
#pragma unroll
                for (int jj = 0; jj < W / 4; ++jj)
                    st_k4<128>(tP, R, c0 + 4 * jj, make_float4(p[4 * jj], p[4 * jj + 1], p[4 * jj + 2], p[4 * jj + 3]));
            }
            fence_async_smem();
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;
        if (issuer) {
            if (lane == 0) {
                tc_fence_after_sync();
                issue<128, 128, false, true, 128, T>(tmem + aO, kdesc<128>(tP), mdesc<T>(tV), true);           // + P V
                mma_commit(barO);
                // once everything has completed the state tile is free for the next pair
                if (mbar_wait(barO, parity, status) && next < npairs) fetch_states(tS, states, next, total, barS);
            }
        } else {
            // the tensor pipe is busy for a while: a good moment to start the next pair's loads
            if (next < npairs) load_raw(raw, q, k, v, gate, g, nit);
            ok = mbar_wait(barO, parity, status);
            if (ok) {
                tc_fence_after_sync();
                float o[W];
                tmem_ld(tmem + lane_base + aO + (uint32_t)(64 * half_r + c0), o);
                store16(reinterpret_cast<TO *>(stage + R * kOutPitch) + c0, o);
            }
            tc_fence_before_sync();
            sync_group(NT);
            if (ok) {
                // coalesced stores of the staged rows: 16 bytes per thread
                constexpr int PER_ROW = 64 * (int)sizeof(TO) / 16;
#pragma unroll
                for (int i = 0; i < PER_ROW / 4; ++i) {
                    const int u = threadIdx.x + NT * i, rr = u / PER_ROW, piece = u % PER_ROW;
                    const Item it = pick(cur[0], cur[1], rr >> 6);
                    const int tr = item_token(g, it, rr & 63);
                    if (tr >= 0)
                        *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(out) + tok_offset(g, it.b, tr, it.h, DV) * sizeof(TO) + piece * 16) =
                            *reinterpret_cast<const uint4 *>(stage + rr * kOutPitch + piece * 16);
                }
            }
        }
        parity ^= 1;
        cur[0] = nit[0];
        cur[1] = nit[1];
    }
    if (!ok) mbar_wait(barS, parity, status);      // let a state copy still in flight land before the CTA's memory goes away
    teardown(ctl, kCols);
}

constexpr size_t out_smem()
{
    return 1024 + 4 * (size_t)kTileK + kTileM + sizeof(float) * (2 * T * kLamPitch + 128 + NT) + sizeof(Control);
}

template <typename TO>
dig_status launch_typed(const GlaArgs &a, const Workspace &w, int sm_count, int *status)
{
    const Geom &g = a.g;
    const int total = g.B * g.H * g.N, npairs = (total + 1) / 2;
    auto kern = tc_out_pair<TO>;
    constexpr size_t smem = out_smem();
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DIG_ERR_CUDA;
    const int grid = npairs < sm_count ? npairs : sm_count;
    KernelTimer t(KID_TC_OUT, a.stream);
    launch_pdl(kern, dim3(grid), dim3(NTA), smem, a.stream, (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v,
               a.gate, (const float *)w.states, (TO *)a.out, status, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

dig_status launch_tc_out(const GlaArgs &a, const Workspace &w, int sm_count, int *status)
{
    return a.dtype == DIG_BF16 ? launch_typed<bf16>(a, w, sm_count, status) : launch_typed<float>(a, w, sm_count, status);
}

}  // namespace dig
