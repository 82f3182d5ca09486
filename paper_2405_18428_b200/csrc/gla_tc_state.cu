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
// the tensor pipe.  Results are staged in shared memory in tile order and leave as one 16 KB bulk
// copy (cp.async.bulk) per chunk and matrix.
#include "tc_tiles.cuh"

namespace dig {
namespace {

using namespace tc;

constexpr int kPairTile = T * 128 * 4;        // bytes of one 64 x 128 M-format tile

template <int NT, bool BWD>
struct StateRaw {
    static constexpr int NROW = 1024 / NT;    // (row, 8-column) pieces per thread over both chunks
    uint4 k[NROW], v[NROW], q[BWD ? NROW : 1], d[BWD ? NROW : 1];
    float4 g0[NROW], g1[NROW];                // the gates of the same 8 columns
};

// Piece i of this thread: chunk half, token row and first column (8 lanes cover one 128-byte bf16 row).
template <int NT>
__device__ __forceinline__ void piece_of(int i, int &half, int &row, int &col)
{
    const int u = threadIdx.x + NT * i;
    half = u >> 9; row = (u >> 3) & 63; col = (u & 7) * 8;
}

template <int NT, bool BWD>
__device__ __forceinline__ void load_raw(StateRaw<NT, BWD> &r, const bf16 *q, const bf16 *k, const bf16 *v,
                                         const bf16 *d_out, const float *gate, const Geom &g, const Item &ia, const Item &ib)
{
#pragma unroll
    for (int i = 0; i < StateRaw<NT, BWD>::NROW; ++i) {
        int half, row, col;
        piece_of<NT>(i, half, row, col);
        const size_t off = row_offset(g, pick(ia, ib, half), row) + col;
        r.k[i] = ldg16(k + off);
        r.v[i] = ldg16(v + off);
        if (BWD) {
            r.q[i] = ldg16(q + off);
            r.d[i] = ldg16(d_out + off);
        }
        const int fl = col >= 32 ? 4 : 0;     // flipped lanes hold their upper four columns first
        r.g0[i] = ldg16(gate + off + fl);
        r.g1[i] = ldg16(gate + off + 4 - fl);
    }
}

template <int NT, bool BWD>
__global__ void __launch_bounds__(NT, BWD ? 1 : 2)
tc_state_pair(const bf16 *__restrict__ q, const bf16 *__restrict__ k, const bf16 *__restrict__ v,
              const float *__restrict__ gate, const bf16 *__restrict__ d_out, float *__restrict__ states,
              float *__restrict__ gamma, float *__restrict__ dstates, int *status, Geom g)
{
    constexpr int W = 64 / (NT / 128);        // accumulator columns per thread
    constexpr int NROW = StateRaw<NT, BWD>::NROW;
    extern __shared__ char smem_raw[];
    char *base = align1024(smem_raw);
    char *tKh = base, *tV = base + kPairTile, *tQ = base + 2 * kPairTile, *tG = base + 3 * kPairTile;
    // once the products have completed, their operand tiles stage the results: chunk a / b of U in
    // the two halves of the first tile, of W in the second
    char *stage = base;
    float *sLam = reinterpret_cast<float *>(base + (BWD ? 4 : 2) * kPairTile);
    float *sLast = sLam + 2 * T * kLamPitch, *sTot = sLast + 128;
    Control *ctl = reinterpret_cast<Control *>(sTot + NT);
    constexpr uint32_t kCols = BWD ? 256 : 128;
    setup(ctl, 1, kCols);
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const uint32_t tmem = ctl->tmem_base;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int R = 32 * (warp & 3) + lane, half_r = R >> 6, r = R & 63, c0 = W * (warp >> 2);

    const int total = g.B * g.H * g.N, npairs = (total + 1) / 2;
    StateRaw<NT, BWD> raw;
    int pair = blockIdx.x;
    Item ca = item_of(g, 2 * pair, total), cb = item_of(g, 2 * pair + 1, total);
    if (pair < npairs) load_raw<NT, BWD>(raw, q, k, v, d_out, gate, g, ca, cb);
    uint32_t parity = 0;
    for (; pair < npairs; pair += gridDim.x) {
        const int next = pair + gridDim.x;
        const Item na = item_of(g, 2 * next, total), nb = item_of(g, 2 * next + 1, total);
        // the previous pair's staged states have been read by the bulk stores
        if (threadIdx.x == 0) bulk_wait_read();
        __syncthreads();
        // gates -> shared memory (log2 units, zero for rows past the end), prefix sums down each chunk
#pragma unroll
        for (int i = 0; i < NROW; ++i) {
            int half, row, col;
            piece_of<NT>(i, half, row, col);
            const Item ci = pick(ca, cb, half);
            const float sc = (ci.valid && ci.chunk * T + row < g.L) ? kLog2e : 0.f;
            float *dst = sLam + (64 * half + row) * kLamPitch + col;
            const int fl = col >= 32 ? 4 : 0;
            *reinterpret_cast<float4 *>(dst + fl) = make_float4(raw.g0[i].x * sc, raw.g0[i].y * sc, raw.g0[i].z * sc, raw.g0[i].w * sc);
            *reinterpret_cast<float4 *>(dst + 4 - fl) = make_float4(raw.g1[i].x * sc, raw.g1[i].y * sc, raw.g1[i].z * sc, raw.g1[i].w * sc);
        }
        __syncthreads();
        gate_prefix<NT, 2>(sLam, sLast, sTot);
        if (threadIdx.x < 128) {
            const int id = 2 * pair + (threadIdx.x >> 6);
            if (id < total) gamma[(size_t)id * DK + (threadIdx.x & 63)] = ex2(sLast[threadIdx.x]);
        }
        // operands
#pragma unroll
        for (int i = 0; i < NROW; ++i) {
            int half, row, col;
            piece_of<NT>(i, half, row, col);
            const bool flip = col >= 32;
            const Item ci = pick(ca, cb, half);
            const bool keep = ci.valid && ci.chunk * T + row < g.L;
            float lam[8], x[8];
            read_lam8(sLam, 64 * half + row, col, lam, flip);
            float last[8];
            read_lam8(sLast, 0, 64 * half + col, last, flip);       // chunk totals of the same columns
            unpack8(raw.k[i], x, keep, flip);
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] *= ex2(last[e] - lam[e]);
            st_m8<T>(tKh, row, 64 * half + col, x, flip);
            unpack8(raw.v[i], x, keep, flip);
            st_m8<T, false>(tV, row, 64 * half + col, x, flip);
            if (BWD) {
                unpack8(raw.q[i], x, keep, flip);
#pragma unroll
                for (int e = 0; e < 8; ++e) x[e] *= ex2(lam[e]);
                st_m8<T>(tQ, row, 64 * half + col, x, flip);
                unpack8(raw.d[i], x, keep, flip);
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
        if (next < npairs) load_raw<NT, BWD>(raw, q, k, v, d_out, gate, g, na, nb);
        const bool ok = mbar_wait(&ctl->bar[0], parity, status);
        parity ^= 1;
        if (ok) {
            // accumulators -> staging, in the tile order the workspace keeps (the layout of store_swizzled)
            tc_fence_after_sync();
            float acc[W];
            tmem_ld(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(64 * half_r + c0), acc);
            store_swizzled(reinterpret_cast<float *>(stage + half_r * (DK * DV * 4)), r, c0, acc);
            if (BWD) {
                tmem_ld(tmem + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(128 + 64 * half_r + c0), acc);
                store_swizzled(reinterpret_cast<float *>(stage + kPairTile + half_r * (DK * DV * 4)), r, c0, acc);
            }
        }
        fence_async_smem();
        tc_fence_before_sync();
        if (!__syncthreads_and(ok)) break;       // a wait gave up: every thread leaves together
        tc_fence_after_sync();
        if (threadIdx.x == 0) {
            // one 16 KB bulk store per chunk and matrix
            for (int half = 0; half < 2; ++half) {
                const int id = 2 * pair + half;
                if (id >= total) break;
                bulk_s2g(states + (size_t)id * (DK * DV), stage + half * (DK * DV * 4), DK * DV * 4);
                if (BWD) bulk_s2g(dstates + (size_t)id * (DK * DV), stage + kPairTile + half * (DK * DV * 4), DK * DV * 4);
            }
            bulk_commit();
        }
        ca = na;
        cb = nb;
    }
    if (threadIdx.x == 0) bulk_wait_all();
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
        launch_pdl(kern, dim3(grid), dim3(NT), smem, a.stream, (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v,
                   a.gate, (const bf16 *)a.d_out, w.states, w.gamma, w.dstates, status, g);
    } else {
        constexpr int NT = 256;           // 100 KB of shared memory: two CTAs per SM overlap each other's phases
        auto kern = tc_state_pair<NT, false>;
        constexpr size_t smem = state_smem<NT, false>();
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return DIG_ERR_CUDA;
        const int grid = npairs < 2 * sm_count ? npairs : 2 * sm_count;
        KernelTimer t(KID_TC_STATE, a.stream);
        launch_pdl(kern, dim3(grid), dim3(NT), smem, a.stream, (const bf16 *)a.q, (const bf16 *)a.k, (const bf16 *)a.v,
                   a.gate, (const bf16 *)nullptr, w.states, w.gamma, (float *)nullptr, status, g);
    }
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
