// Scans over the per-chunk states of chunkwise gated linear attention (Section 3.5 splits the
// sequence into chunks; the recurrence of Eq. attn_gla then links the chunks):
//   forward :  S_[i+1] = diag(gamma_i) S_[i] + U_i,  S_[0] = 0      (U_i in, S_[i] out, in place)
//   backward:  D_[i-1] = diag(gamma_i) D_[i] + W_i,  D_[N-1] = 0    (W_i in, D_[i] out, in place)
//              carry_i[c] = sum_e S_[i+1][c][e] * D_[i][c][e]       (0 for the last chunk)
// S_[i] is the state entering chunk i, D_[i] the gradient of the loss with respect to the state
// leaving chunk i, and carry_i the part of the gate gradient that tokens of later chunks
// contribute to every token of chunk i.  Plain fp32 FMAs; the work is a dependent chain over
// the N chunks per element, so loads are issued a few chunks ahead of their use.
#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int kScanThreads = 128;
constexpr int kAhead = 4;

__global__ void __launch_bounds__(kScanThreads)
state_scan_fwd(float *__restrict__ states, const float *__restrict__ gamma, int N, int dk, int dv)
{
    const int elem = blockIdx.x * kScanThreads + threadIdx.x;
    if (elem >= dk * dv) return;
    const int c = elem / dv;
    float *st = states + (size_t)blockIdx.y * N * dk * dv + elem;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + c;
    const size_t sstride = (size_t)dk * dv;
    float run = 0.f;
    int i = 0;
    for (; i + kAhead <= N; i += kAhead) {
        float u[kAhead], g[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            u[j] = st[(size_t)(i + j) * sstride];
            g[j] = gm[(size_t)(i + j) * dk];
        }
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            st[(size_t)(i + j) * sstride] = run;
            run = fmaf(g[j], run, u[j]);
        }
    }
    for (; i < N; ++i) {
        const float u = st[(size_t)i * sstride], g = gm[(size_t)i * dk];
        st[(size_t)i * sstride] = run;
        run = fmaf(g, run, u);
    }
}

// One warp per key channel c; lanes stride over the value channels.
constexpr int kRowsPerBlock = 4;
constexpr int kMaxPerLane = 4;     // d_v <= 128

__global__ void __launch_bounds__(32 * kRowsPerBlock)
state_scan_bwd(const float *__restrict__ states, float *__restrict__ dstates,
               const float *__restrict__ gamma, float *__restrict__ carry, int N, int dk, int dv)
{
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (c >= dk) return;
    const size_t sstride = (size_t)dk * dv;
    const size_t base = (size_t)blockIdx.y * N * sstride + (size_t)c * dv;
    const float *S = states + base;
    float *D = dstates + base;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + c;
    float *cr = carry + (size_t)blockIdx.y * N * dk + c;
    float run[kMaxPerLane];
#pragma unroll
    for (int r = 0; r < kMaxPerLane; ++r) run[r] = 0.f;
    for (int i = N - 1; i >= 0; --i) {
        float w[kMaxPerLane], sn[kMaxPerLane];
        const float g = gm[(size_t)i * dk];
#pragma unroll
        for (int r = 0; r < kMaxPerLane; ++r) {
            const int e = lane + 32 * r;
            w[r] = (e < dv) ? D[(size_t)i * sstride + e] : 0.f;
            sn[r] = (e < dv && i + 1 < N) ? S[(size_t)(i + 1) * sstride + e] : 0.f;
        }
        float dot = 0.f;
#pragma unroll
        for (int r = 0; r < kMaxPerLane; ++r) {
            const int e = lane + 32 * r;
            if (e < dv) D[(size_t)i * sstride + e] = run[r];
            dot = fmaf(sn[r], run[r], dot);
            run[r] = fmaf(g, run[r], w[r]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
        if (lane == 0) cr[(size_t)i * dk] = dot;
    }
}

}  // namespace

dig_status launch_state_scan_fwd(const Workspace &w, const Geom &g, cudaStream_t s)
{
    const dim3 grid((g.dk * g.dv + kScanThreads - 1) / kScanThreads, g.B * g.H);
    KernelTimer t(KID_SCAN_FWD, s);
    state_scan_fwd<<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, g.N, g.dk, g.dv);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_state_scan_bwd(const Workspace &w, const Geom &g, cudaStream_t s)
{
    const dim3 grid((g.dk + kRowsPerBlock - 1) / kRowsPerBlock, g.B * g.H);
    KernelTimer t(KID_SCAN_BWD, s);
    state_scan_bwd<<<grid, 32 * kRowsPerBlock, 0, s>>>(w.states, w.dstates, w.gamma, w.carry, g.N,
                                                       g.dk, g.dv);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
