// Scans over the per-chunk states of chunkwise gated linear attention (Section 3.5 splits the
// sequence into chunks; the recurrence of Eq. attn_gla then links the chunks):
//   forward :  S_[i+1] = diag(gamma_i) S_[i] + U_i,  S_[0] = 0      (U_i in, S_[i] out, in place)
//   backward:  D_[i-1] = diag(gamma_i) D_[i] + W_i,  D_[N-1] = 0    (W_i in, D_[i] out, in place)
//              carry_i[c] = sum_e S_[i+1][c][e] * D_[i][c][e]       (0 for the last chunk)
// S_[i] is the state entering chunk i, D_[i] the gradient of the loss with respect to the state
// leaving chunk i, and carry_i the part of the gate gradient that tokens of later chunks
// contribute to every token of chunk i.  Plain fp32 FMAs; the work is a dependent chain over
// the N chunks per element, so loads are issued a few chunks ahead of their use.
// Optional state arguments ([B*H][d_k][d_v] row-major fp32, null = zero / not wanted): the forward scan
// starts from s_in and hands out the state after the last chunk; the backward scan starts from the
// gradient with respect to that final state and hands out the gradient with respect to s_in.
#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int kScanThreads = 128;
constexpr int kAhead = 16;

__device__ __forceinline__ float round_tf32(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xffffe000u);
}
__device__ __forceinline__ float4 round4_tf32(float4 v)
{
    return make_float4(round_tf32(v.x), round_tf32(v.y), round_tf32(v.z), round_tf32(v.w));
}

// One thread per 4 consecutive state elements; states are [d_k][d_v] row-major, the decay is indexed
// by the row.  The loads of a batch of kAhead chunks do not depend on the running value, so they are
// all in flight before the short dependent chain of FMAs runs.
// TF32: the stored states are rounded to tf32 (warp-MMA family); the running value is not.
template <bool TF32 = false>
__global__ void __launch_bounds__(kScanThreads)
state_scan_fwd(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ s_in,
               float *__restrict__ s_final, int N, int dk, int dv)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int e4 = blockIdx.x * kScanThreads + threadIdx.x;          // float4 index inside one state
    if (e4 * 4 >= dk * dv) return;
    const int row = (e4 * 4) / dv, col = (e4 * 4) - row * dv;
    float4 *st = reinterpret_cast<float4 *>(states + (size_t)blockIdx.y * N * dk * dv) + e4;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + row;
    const size_t sstride = (size_t)dk * dv / 4;
    float4 run = make_float4(0.f, 0.f, 0.f, 0.f);
    const size_t io = (size_t)blockIdx.y * dk * dv + (size_t)row * dv + col, ios = 1;
    if (s_in != nullptr) run = make_float4(s_in[io], s_in[io + ios], s_in[io + 2 * ios], s_in[io + 3 * ios]);
    for (int i = 0; i < N; i += kAhead) {
        float4 u[kAhead], g[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                u[j] = st[(size_t)(i + j) * sstride];
                g[j].x = g[j].y = g[j].z = g[j].w = gm[(size_t)(i + j) * dk];
            }
        }
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                st[(size_t)(i + j) * sstride] = TF32 ? round4_tf32(run) : run;
                run.x = fmaf(g[j].x, run.x, u[j].x);
                run.y = fmaf(g[j].y, run.y, u[j].y);
                run.z = fmaf(g[j].z, run.z, u[j].z);
                run.w = fmaf(g[j].w, run.w, u[j].w);
            }
        }
    }
    if (s_final != nullptr) {
        s_final[io] = run.x;
        s_final[io + ios] = run.y;
        s_final[io + 2 * ios] = run.z;
        s_final[io + 3 * ios] = run.w;
    }
}

// The same scan with one element per thread and 16 chunks of loads in flight: four times the threads
// of the kernel above, for calls with so few (batch, head) sequences that float4 threads would leave
// most SMs idle and too few loads in flight (long sequences of a small batch).
constexpr int kScan1Threads = 256, kAhead1 = 16;
template <bool TF32>
__global__ void __launch_bounds__(kScan1Threads)
state_scan_fwd1(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ s_in,
                float *__restrict__ s_final, int N, int dk, int dv)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int e = blockIdx.x * kScan1Threads + threadIdx.x;          // element index inside one stored state
    if (e >= dk * dv) return;
    const int row = e / dv, col = e - row * dv;
    float *st = states + (size_t)blockIdx.y * N * dk * dv + e;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + row;
    const size_t sstride = (size_t)dk * dv;
    const size_t io = (size_t)blockIdx.y * dk * dv + (size_t)row * dv + col;
    float run = s_in != nullptr ? s_in[io] : 0.f;
    for (int i = 0; i < N; i += kAhead1) {
        float u[kAhead1], g[kAhead1];
        const float *pu = st;
        const float *pg = gm;
#pragma unroll
        for (int j = 0; j < kAhead1; ++j) {
            if (i + j < N) {
                u[j] = *pu;
                g[j] = *pg;
            }
            pu += sstride;
            pg += dk;
        }
#pragma unroll
        for (int j = 0; j < kAhead1; ++j) {
            if (i + j < N) {
                *st = TF32 ? round_tf32(run) : run;
                run = fmaf(g[j], run, u[j]);
            }
            st += sstride;
        }
        gm += (size_t)kAhead1 * dk;
    }
    if (s_final != nullptr) s_final[io] = run;
}

// One warp per key channel c; lanes stride over the value channels.
// TF32: dstates receives diag(gamma_i) D_[i] rounded to tf32, the form the warp-MMA gradient kernel
// multiplies with, instead of D_[i].
constexpr int kRowsPerBlock = 4;
constexpr int kMaxPerLane = 4;     // d_v <= 128

template <bool TF32>
__global__ void __launch_bounds__(32 * kRowsPerBlock)
state_scan_bwd(const float *__restrict__ states, float *__restrict__ dstates,
               const float *__restrict__ gamma, float *__restrict__ carry, const float *__restrict__ s_final,
               const float *__restrict__ ds_out, float *__restrict__ ds_in, int N, int dk, int dv)
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
    const size_t io = ((size_t)blockIdx.y * dk + c) * dv;
#pragma unroll
    for (int r = 0; r < kMaxPerLane; ++r) {
        const int e = lane + 32 * r;
        run[r] = (ds_out != nullptr && e < dv) ? ds_out[io + e] : 0.f;
    }
    // kLook chunks are loaded ahead of the recurrence, so the walk pays the latency of global memory
    // once per kLook chunks and not once per chunk
    constexpr int kLook = 8;
    for (int i = N - 1; i >= 0; i -= kLook) {
        float w[kLook][kMaxPerLane], sn[kLook][kMaxPerLane], g[kLook];
#pragma unroll
        for (int j = 0; j < kLook; ++j) {
            const int ch = i - j;
            g[j] = 0.f;
            if (ch >= 0) g[j] = gm[(size_t)ch * dk];
#pragma unroll
            for (int r = 0; r < kMaxPerLane; ++r) {
                const int e = lane + 32 * r;
                w[j][r] = (ch >= 0 && e < dv) ? D[(size_t)ch * sstride + e] : 0.f;
                sn[j][r] = 0.f;          // the state leaving chunk ch: the next chunk's entry, or the final state
                if (ch >= 0 && e < dv) {
                    if (ch + 1 < N) sn[j][r] = S[(size_t)(ch + 1) * sstride + e];
                    else if (ds_out != nullptr) sn[j][r] = s_final[io + e];
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kLook; ++j) {
            const int ch = i - j;
            if (ch < 0) break;          // uniform over the warp
            float dot = 0.f;
#pragma unroll
            for (int r = 0; r < kMaxPerLane; ++r) {
                const int e = lane + 32 * r;
                if (e < dv) D[(size_t)ch * sstride + e] = TF32 ? round_tf32(g[j] * run[r]) : run[r];
                dot = fmaf(sn[j][r], run[r], dot);
                run[r] = fmaf(g[j], run[r], w[j][r]);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
            if (lane == 0) cr[(size_t)ch * dk] = dot;
        }
    }
    if (ds_in != nullptr) {
#pragma unroll
        for (int r = 0; r < kMaxPerLane; ++r) {
            const int e = lane + 32 * r;
            if (e < dv) ds_in[io + e] = run[r];
        }
    }
}

// ---- the same scans with the value-channel gate (full gate G = alpha^T beta of Eq. gate_gla) ---------
// The state decays along its rows by gamma (key channels) and along its columns by gamma_v (value
// channels): S_[i+1] = diag(gamma_i) S_[i] diag(gamma_v_i) + U_i, and the mirror image for D.  Row-major
// states only (warp-MMA family); with `tf32` the stored states and diag(gamma) D diag(gamma_v) are rounded to tf32.
__global__ void __launch_bounds__(kScanThreads)
state_scan_fwd_beta(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ gamma_v,
                    float *__restrict__ s_final, int N, int dk, int dv, bool tf32)
{
    const int e4 = blockIdx.x * kScanThreads + threadIdx.x;
    if (e4 * 4 >= dk * dv) return;
    const int row = (e4 * 4) / dv, col = (e4 * 4) - row * dv;
    float4 *st = reinterpret_cast<float4 *>(states + (size_t)blockIdx.y * N * dk * dv) + e4;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + row;
    const float *gv = gamma_v + (size_t)blockIdx.y * N * dv + col;
    const size_t sstride = (size_t)dk * dv / 4;
    float4 run = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i = 0; i < N; i += kAhead) {
        float4 u[kAhead], g[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                u[j] = st[(size_t)(i + j) * sstride];
                const float gr = gm[(size_t)(i + j) * dk];
                const float4 gc = *reinterpret_cast<const float4 *>(gv + (size_t)(i + j) * dv);
                g[j] = make_float4(gr * gc.x, gr * gc.y, gr * gc.z, gr * gc.w);
            }
        }
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                st[(size_t)(i + j) * sstride] = tf32 ? round4_tf32(run) : run;
                run.x = fmaf(g[j].x, run.x, u[j].x);
                run.y = fmaf(g[j].y, run.y, u[j].y);
                run.z = fmaf(g[j].z, run.z, u[j].z);
                run.w = fmaf(g[j].w, run.w, u[j].w);
            }
        }
    }
    if (s_final != nullptr) *reinterpret_cast<float4 *>(s_final + (size_t)blockIdx.y * dk * dv + (size_t)e4 * 4) = run;
}

__global__ void __launch_bounds__(32 * kRowsPerBlock)
state_scan_bwd_beta(const float *__restrict__ states, float *__restrict__ dstates, const float *__restrict__ gamma,
                    const float *__restrict__ gamma_v, float *__restrict__ carry, int N, int dk, int dv, bool tf32)
{
    const int lane = threadIdx.x & 31;
    const int c = blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (c >= dk) return;
    const size_t sstride = (size_t)dk * dv;
    const size_t base = (size_t)blockIdx.y * N * sstride + (size_t)c * dv;
    const float *S = states + base;
    float *D = dstates + base;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + c;
    const float *gv = gamma_v + (size_t)blockIdx.y * N * dv;
    float *cr = carry + (size_t)blockIdx.y * N * dk + c;
    float run[kMaxPerLane];
#pragma unroll
    for (int r = 0; r < kMaxPerLane; ++r) run[r] = 0.f;
    constexpr int kLook = 4;
    for (int i = N - 1; i >= 0; i -= kLook) {
        float w[kLook][kMaxPerLane], sn[kLook][kMaxPerLane], g[kLook][kMaxPerLane];
#pragma unroll
        for (int j = 0; j < kLook; ++j) {
            const int ch = i - j;
            const float gr = ch >= 0 ? gm[(size_t)ch * dk] : 0.f;
#pragma unroll
            for (int r = 0; r < kMaxPerLane; ++r) {
                const int e = lane + 32 * r;
                const bool on = ch >= 0 && e < dv;
                w[j][r] = on ? D[(size_t)ch * sstride + e] : 0.f;
                g[j][r] = on ? gr * gv[(size_t)ch * dv + e] : 0.f;
                sn[j][r] = (on && ch + 1 < N) ? S[(size_t)(ch + 1) * sstride + e] : 0.f;
            }
        }
#pragma unroll
        for (int j = 0; j < kLook; ++j) {
            const int ch = i - j;
            if (ch < 0) break;          // uniform over the warp
            float dot = 0.f;
#pragma unroll
            for (int r = 0; r < kMaxPerLane; ++r) {
                const int e = lane + 32 * r;
                if (e < dv) D[(size_t)ch * sstride + e] = tf32 ? round_tf32(g[j][r] * run[r]) : g[j][r] * run[r];
                dot = fmaf(sn[j][r], run[r], dot);
                run[r] = fmaf(g[j][r], run[r], w[j][r]);
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
            if (lane == 0) cr[(size_t)ch * dk] = dot;
        }
    }
}

// Gate gradient of the value-channel gate across chunks.  xtot[i][e] holds chunk i's total of
// (o*do - v*dv); it is turned in place into the sum over the later chunks (what every token of chunk
// i still has to receive), one thread per (sequence, value channel).
__global__ void __launch_bounds__(128)
beta_suffix_totals(float *__restrict__ xtot, int N, int dv, int total)
{
    const int idx = blockIdx.x * 128 + threadIdx.x;
    if (idx >= total) return;
    const int bh = idx / dv, e = idx - bh * dv;
    float *x = xtot + (size_t)bh * N * dv + e;
    float run = 0.f;
    for (int i = N - 1; i >= 0; --i) {
        const float t = x[(size_t)i * dv];
        x[(size_t)i * dv] = run;
        run += t;
    }
}

// dbgate[token][e] += what later chunks contribute; one thread per 4 value channels of a scan position.
__global__ void __launch_bounds__(256)
beta_add_carry(float *__restrict__ dbgate, const float *__restrict__ xtot, Geom g)
{
    const int per_row = g.dv >> 2;
    const long long idx = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long total = (long long)g.B * g.H * g.L * per_row;
    if (idx >= total) return;
    const int e = (int)(idx % per_row) << 2;
    const long long r = idx / per_row;
    const int p = (int)(r % g.L);
    const int bh = (int)(r / g.L), b = bh / g.H, h = bh - b * g.H;
    const int chunk = p / g.C;
    const float4 add = *reinterpret_cast<const float4 *>(xtot + ((size_t)bh * g.N + chunk) * g.dv + e);
    float4 *dst = reinterpret_cast<float4 *>(dbgate + tok_offset(g, b, scan_token(p, g.dir, g.gh, g.gw, g.L), h, g.dv) + e);
    float4 v = *dst;
    v.x += add.x; v.y += add.y; v.z += add.z; v.w += add.w;
    *dst = v;
}

}  // namespace

dig_status launch_state_scan_fwd(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio, bool tf32)
{
    const dim3 grid((g.dk * g.dv / 4 + kScanThreads - 1) / kScanThreads, g.B * g.H);
    // the state after the last chunk goes to the caller if asked for, else to the workspace block the
    // backward scan reads it from (null in a forward-only workspace)
    float *fin = sio.s_out != nullptr ? sio.s_out : w.sfinal;
    KernelTimer t(KID_SCAN_FWD, s);
    if ((long long)grid.x * grid.y * kScanThreads < 16384) {       // few sequences: one element per thread
        const dim3 grid1((g.dk * g.dv + kScan1Threads - 1) / kScan1Threads, g.B * g.H);
        if (tf32)
            state_scan_fwd1<true><<<grid1, kScan1Threads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
        else
            state_scan_fwd1<false><<<grid1, kScan1Threads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
        return cuda_ok(cudaGetLastError());
    }
    if (tf32)
        state_scan_fwd<true><<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
    else
        state_scan_fwd<false><<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
    return cuda_ok(cudaGetLastError());
}

// Needs the final state in w.sfinal (left there by launch_state_scan_fwd on a backward workspace).
dig_status launch_state_scan_bwd(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio, bool tf32)
{
    const dim3 grid((g.dk + kRowsPerBlock - 1) / kRowsPerBlock, g.B * g.H);
    KernelTimer t(KID_SCAN_BWD, s);
    if (tf32)
        state_scan_bwd<true><<<grid, 32 * kRowsPerBlock, 0, s>>>(w.states, w.dstates, w.gamma, w.carry, w.sfinal, sio.ds_out,
                                                                 sio.ds_in, g.N, g.dk, g.dv);
    else
        state_scan_bwd<false><<<grid, 32 * kRowsPerBlock, 0, s>>>(w.states, w.dstates, w.gamma, w.carry, w.sfinal, sio.ds_out,
                                                                  sio.ds_in, g.N, g.dk, g.dv);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_state_scan_fwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s, bool tf32)
{
    const dim3 grid((g.dk * g.dv / 4 + kScanThreads - 1) / kScanThreads, g.B * g.H);
    KernelTimer t(KID_SCAN_FWD, s);
    state_scan_fwd_beta<<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, gamma_v, w.sfinal, g.N, g.dk, g.dv, tf32);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_state_scan_bwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s, bool tf32)
{
    const dim3 grid((g.dk + kRowsPerBlock - 1) / kRowsPerBlock, g.B * g.H);
    KernelTimer t(KID_SCAN_BWD, s);
    state_scan_bwd_beta<<<grid, 32 * kRowsPerBlock, 0, s>>>(w.states, w.dstates, w.gamma, gamma_v, w.carry, g.N, g.dk, g.dv, tf32);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_beta_carry(float *dbgate, float *xtot, const Geom &g, cudaStream_t s)
{
    KernelTimer t(KID_SCAN_BWD, s);
    const int total = g.B * g.H * g.dv;
    beta_suffix_totals<<<(total + 127) / 128, 128, 0, s>>>(xtot, g.N, g.dv, total);
    if (cudaGetLastError() != cudaSuccess) return DIG_ERR_CUDA;
    const long long n = (long long)g.B * g.H * g.L * (g.dv >> 2);
    beta_add_carry<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(dbgate, xtot, g);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
