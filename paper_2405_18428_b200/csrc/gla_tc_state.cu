// Tensor-core kernel for the chunk-local state contributions of chunkwise gated linear attention
// (Eq. attn_gla split into chunks, Section 3.5):
//   forward pass : U^T = V^T Kh          per chunk, a [d_v][d_k] matrix
//   backward pass: U   = Kh^T V,  W = Qt^T dO,     [d_k][d_v] matrices
// each stored in the swizzled operand-tile order of the kernels that consume the scanned states,
// with Kh = k*exp(Lam_last - Lam), Qt = q*exp(Lam), Lam the in-chunk cumulative gate, and
// gamma = exp(Lam_last) per chunk.
//
// A CTA works on two chunks at a time.  Their operand tiles sit side by side in M-format tiles of
// 64 token rows x 128 columns, so one tcgen05.mma sequence with M = N = 128 (8 instructions: an
// instruction costs the same ~60 cycles whether it is 64 or 128 wide) yields both chunks' products
// on the diagonal blocks of a 128 x 128 accumulator; the off-diagonal blocks are never read.
// CTAs are persistent and prefetch the next pair's rows into registers while the current pair is in
// the tensor pipe.
#include "tc_tiles.cuh"

namespace dig {
namespace {

using namespace tc;

constexpr int kPairTile = T * 128 * 4;        // bytes of one 64 x 128 M-format tile

template <int NT, bool BWD>
struct StateRaw {
    static constexpr int NROW = 1024 / NT;    // 16-byte row pieces per tensor per thread (both chunks)
    static constexpr int NG = 2048 / NT;      // float4 gate pieces per thread (both chunks)
    uint4 k[NROW], v[NROW], q[BWD ? NROW : 1], d[BWD ? NROW : 1];
    float4 g[NG];
};

template <int NT, bool BWD>
__device__ __forceinline__ void load_raw(StateRaw<NT, BWD> &r, const bf16 *q, const bf16 *k, const bf16 *v,
                                         const bf16 *d_out, const float *gate, const Geom &g, int pair, int total)
{
    const Item it[2] = {item_of(g, 2 * pair, total), item_of(g, 2 * pair + 1, total)};
#pragma unroll
    for (int i = 0; i < StateRaw<NT, BWD>::NROW; ++i) {
        const int u = threadIdx.x + NT * i, half = u >> 9, row = (u >> 3) & 63, col = (u & 7) * 8;
        const int tok = item_token(g, it[half], row);
        r.k[i] = ld_row8(k, g, it[half].b, tok, it[half].h, DK, col);
        r.v[i] = ld_row8(v, g, it[half].b, tok, it[half].h, DV, col);
        if (BWD) {
            r.q[i] = ld_row8(q, g, it[half].b, tok, it[half].h, DK, col);
            r.d[i] = ld_row8(d_out, g, it[half].b, tok, it[half].h, DV, col);
        }
    }
#pragma unroll
    for (int i = 0; i < StateRaw<NT, BWD>::NG; ++i) {
        const int u = threadIdx.x + NT * i, half = u >> 10, row = (u >> 4) & 63, col = (u & 15) * 4;
        const int tok = item_token(g, it[half], row);
        r.g[i] = ld_row4(gate, g, it[half].b, tok, it[half].h, DK, col);
    }
}

template <int NT, bool BWD>
__global__ void __launch_bounds__(NT)
tc_state_pair(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
              const float *__restrict__ gate, const bf16 *__restrict__ d_out, float *__restrict__ states,
              float *__restrict__ gamma, float *__restrict__ dstates, int *status, Geom g)
{
    constexpr int W = 64 / (NT / 128);        // accumulator columns per thread
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    char *tKh = base, *tV = base + kPairTile, *tQ = base + 2 * kPairTile, *tG = base + 3 * kPairTile;
    float *sLam = reinterpret_cast<float *>(base + (BWD ? 4 : 2) * kPairTile);
    float *sLast = sLam + 2 * T * kLamPitch, *sTot = sLast + 128;
    Control *ctl = reinterpret_cast<Control *>(sTot + NT);
    constexpr uint32_t kCols = BWD ? 256 : 128;
    setup(ctl, 1, kCols);
    const uint32_t tmem = ctl->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = 32 * (warp & 3) + lane, half_r = R >> 6, r = R & 63, c0 = W * (warp >> 2);

    const int total = g.B * g.H * g.N, npairs = (total + 1) / 2;
    StateRaw<NT, BWD> raw;
    int pair = blockIdx.x;
    if (pair < npairs) load_raw<NT, BWD>(raw, q, k, v, d_out, gate, g, pair, total);
    uint32_t parity = 0;
    for (; pair < npairs; pair += gridDim.x) {
        // gates -> shared memory (log2 units, zero for rows past the end), prefix sums down each chunk
#pragma unroll
        for (int i = 0; i < StateRaw<NT, BWD>::NG; ++i) {
            const int u = threadIdx.x + NT * i, row = (u >> 4) & 127, col = (u & 15) * 4;
            const int id = 2 * pair + (row >> 6);
            const float sc = (id < total && (id % g.N) * T + (row & 63) < g.L) ? kLog2e : 0.f;
            const float4 a = raw.g[i];
            *reinterpret_cast<float4 *>(sLam + row * kLamPitch + col) = make_float4(a.x * sc, a.y * sc, a.z * sc, a.w * sc);
        }
        __syncthreads();
        gate_prefix<NT, 2>(sLam, sLast, sTot);
        if (threadIdx.x < 128) {
            const int id = 2 * pair + (threadIdx.x >> 6);
            if (id < total) gamma[(size_t)id * DK + (threadIdx.x & 63)] = ex2(sLast[threadIdx.x]);
        }
        // operands
#pragma unroll
        for (int i = 0; i < StateRaw<NT, BWD>::NROW; ++i) {
            const int u = threadIdx.x + NT * i, half = u >> 9, row = (u >> 3) & 63, j = u & 7, col = j * 8;
            const bool flip = j >= 4;
            const int id = 2 * pair + half;
            const bool keep = id < total && (id % g.N) * T + row < g.L;
            float lam[8], x[8];
            read_lam8(sLam, 64 * half + row, col, lam);
            unpack8(raw.k[i], x, keep);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] *= ex2(sLast[64 * half + col + e] - lam[e]);
            st_m8<T>(tKh, row, 64 * half + col, x, flip);
            unpack8(raw.v[i], x, keep);
            st_m8<T, false>(tV, row, 64 * half + col, x, flip);
            if (BWD) {
                unpack8(raw.q[i], x, keep);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] *= ex2(lam[e]);
                st_m8<T>(tQ, row, 64 * half + col, x, flip);
                unpack8(raw.d[i], x, keep);
                st_m8<T, false>(tG, row, 64 * half + col, x, flip);
            }
        }
        fence_async_smem();
        tc_fence_before_sync();
        __syncthreads();
        if (threadIdx.x == 0) {
            tc_fence_after_sync();
            if (BWD) {
                issue<128, 128, true, true, T, T>(tmem, mdesc<T>(tKh), mdesc<T>(tV), false);          // U   [c][e]
                issue<128, 128, true, true, T, T>(tmem + 128, mdesc<T>(tQ), mdesc<T>(tG), false);     // W   [c][e]
            } else {
                issue<128, 128, true, true, T, T>(tmem, mdesc<T>(tV), mdesc<T>(tKh), false);          // U^T [e][c]
            }
            mma_commit(&ctl->bar[0]);
        }
        const int next = pair + gridDim.x;
        if (next < npairs) load_raw<NT, BWD>(raw, q, k, v, d_out, gate, g, next, total);
        const bool ok = mbar_wait(&ctl->bar[0], parity, status);
        parity ^= 1;
        if (ok) {
            tc_fence_after_sync();
            const int id = 2 * pair + half_r;
            float acc[W];
            tmem_ld(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(64 * half_r + c0), acc);
            if (id < total) store_swizzled(states + (size_t)id * (DK * DV), r, c0, acc);
            if (BWD) {
                tmem_ld(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(128 + 64 * half_r + c0), acc);
                if (id < total) store_swizzled(dstates + (size_t)id * (DK * DV), r, c0, acc);
            }
        }
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;       // a wait gave up: every thread leaves together
        tc_fence_after_sync();
    }
    teardown(ctl, kCols);
}

template <int NT, bool BWD>
constexpr size_t state_smem()
{
    return 1024 + (size_t)(BWD ? 4 : 2) * kPairTile + sizeof(float) * (2 * T * kLamPitch + 128 + NT) + sizeof(Control);
}

}  // namespace

// Launches the chunk-state kernel.  Forward: states receive U^T ([d_v][d_k] per chunk);
// backward: states receive U and dstates W (both [d_k][d_v]); gamma in both cases.
dig_status launch_tc_state(const GlaArgs &a, const Workspace &w, bool backward, int sm_count, int *status)
{
    const Geom &g = a.g;
    const int total = g.B * g.H * g.N, npairs = (total + 1) / 2;
    if (backward) {
        constexpr int NT = 512;
        auto kern = tc_state_pair<NT, true>;
        constexpr size_t smem = state_smem<NT, true>();
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DIG_ERR_CUDA;
        const int grid = npairs < sm_count ? npairs : sm_count;
        KernelTimer t(KID_TC_STATE, a.stream);
        kern<<<grid, NT, smem, a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate,
                                           (const bf16 *)a.d_out, w.states, w.gamma, w.dstates, status, g);
    } else {
        constexpr int NT = 512;
        auto kern = tc_state_pair<NT, false>;
        constexpr size_t smem = state_smem<NT, false>();
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DIG_ERR_CUDA;
        const int grid = npairs < sm_count ? npairs : sm_count;
        KernelTimer t(KID_TC_STATE, a.stream);
        kern<<<grid, NT, smem, a.stream>>>((const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v, a.gate,
                                           nullptr, w.states, w.gamma, nullptr, status, g);
    }
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
