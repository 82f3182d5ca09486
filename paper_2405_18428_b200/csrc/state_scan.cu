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

// One thread per 4 consecutive state elements.  TILES = false: states are [d_k][d_v] row-major,
// decay indexed by the row.  TILES = true (tensor-core forward pass, d_k = d_v = 64): each state is
// stored transposed ([d_v][d_k]) in the swizzled operand-tile order the output kernel copies
// straight into shared memory (two column blocks of 64 rows x 128 bytes, 16-byte pieces of a row
// XOR-ed with row & 7); the decay is indexed by the logical column, and the stored states are
// rounded to tf32 (the running value is not).
// The loads of a batch of kAhead chunks do not depend on the running value, so they are all in
// flight before the short dependent chain of FMAs runs.
// TF32: the stored states are rounded to tf32 although they stay row-major (warp-MMA family).
template <bool TILES, bool TF32 = false>
__global__ void __launch_bounds__(kScanThreads)
state_scan_fwd(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ s_in,
               float *__restrict__ s_final, int N, int dk, int dv)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int e4 = blockIdx.x * kScanThreads + threadIdx.x;          // float4 index inside one state
    if (e4 * 4 >= dk * dv) return;
    int row, col;
    if (TILES) {
        row = (e4 & 511) >> 3;
        col = (e4 >> 9) * 32 + (((e4 & 7) ^ (row & 7)) << 2);
    } else {
        row = (e4 * 4) / dv;
        col = (e4 * 4) - row * dv;
    }
    float4 *st = reinterpret_cast<float4 *>(states + (size_t)blockIdx.y * N * dk * dv) + e4;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + (TILES ? col : row);
    const size_t sstride = (size_t)dk * dv / 4;
    float4 run = make_float4(0.f, 0.f, 0.f, 0.f);
    // this thread's four elements in a row-major [d_k][d_v] state: consecutive (plain layout) or a
    // stride of d_v apart (the transposed tiles hold S[col .. col+3][row])
    const size_t io = (size_t)blockIdx.y * dk * dv + (TILES ? (size_t)col * dv + row : (size_t)row * dv + col);
    const size_t ios = TILES ? (size_t)dv : 1;
    if (s_in != nullptr) run = make_float4(s_in[io], s_in[io + ios], s_in[io + 2 * ios], s_in[io + 3 * ios]);
    for (int i = 0; i < N; i += kAhead) {
        float4 u[kAhead], g[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                u[j] = st[(size_t)(i + j) * sstride];
                if (TILES) g[j] = *reinterpret_cast<const float4 *>(gm + (size_t)(i + j) * dk);
                else g[j].x = g[j].y = g[j].z = g[j].w = gm[(size_t)(i + j) * dk];
            }
        }
#pragma unroll
        for (int j = 0; j < kAhead; ++j) {
            if (i + j < N) {
                st[(size_t)(i + j) * sstride] = (TILES || TF32) ? round4_tf32(run) : run;
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
template <bool TILES, bool TF32>
__global__ void __launch_bounds__(kScan1Threads)
state_scan_fwd1(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ s_in,
                float *__restrict__ s_final, int N, int dk, int dv)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int e = blockIdx.x * kScan1Threads + threadIdx.x;          // element index inside one stored state
    if (e >= dk * dv) return;
    int row, col;
    if (TILES) {
        row = (e & 2047) >> 5;
        col = (e >> 11) * 32 + ((((e & 31) >> 2) ^ (row & 7)) << 2) + (e & 3);
    } else {
        row = e / dv;
        col = e - row * dv;
    }
    float *st = states + (size_t)blockIdx.y * N * dk * dv + e;
    const float *gm = gamma + (size_t)blockIdx.y * N * dk + (TILES ? col : row);
    const size_t sstride = (size_t)dk * dv;
    const size_t io = (size_t)blockIdx.y * dk * dv + (TILES ? (size_t)col * dv + row : (size_t)row * dv + col);
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
                *st = (TILES || TF32) ? round_tf32(run) : run;
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

// Both scans of the tensor-core backward pass in one launch (d_k = d_v = 64).  The per-chunk
// matrices U (in `states`) and W (in `dstates`) are [d_k][d_v] in swizzled tile order; a thread owns
// the same 16-byte piece of one row in both column blocks (8 floats), so the decay index is its row
// and the order of the pieces inside the row does not matter.  It first runs the forward
// recurrence (states <- S_[i], rounded to tf32 for the consumer), then walks back over the chunks:
//   dstates, dstates_m <- diag(gamma_i) D_[i] (rounded to tf32, in the two operand-tile orders),
//   carry_i = row sums of S_[i+1] * D_[i],
// reading back the S values it wrote itself.  Block = 8 rows x 8 pieces; grid (8, B*H).
constexpr int kBack = 8;
__device__ __forceinline__ float4 fma4(float g, float4 r, float4 u)
{
    return make_float4(fmaf(g, r.x, u.x), fmaf(g, r.y, u.y), fmaf(g, r.z, u.z), fmaf(g, r.w, u.w));
}
__global__ void __launch_bounds__(64)
state_scan_bwd_tiles(float *__restrict__ states, float *__restrict__ dstates, float *__restrict__ dstates_m,
                     const float *__restrict__ gamma, float *__restrict__ carry, const float *__restrict__ s_in,
                     const float *__restrict__ ds_out, float *__restrict__ ds_in, int N)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int t = threadIdx.x, c = 8 * blockIdx.x + (t >> 3);
    const size_t base = (size_t)blockIdx.y * N * 4096;
    float4 *S = reinterpret_cast<float4 *>(states + base) + c * 8 + (t & 7);
    float4 *D = reinterpret_cast<float4 *>(dstates + base) + c * 8 + (t & 7);
    // The same values once more in the other tile order (32-byte pieces of a row XOR-ed with row & 3):
    // this thread's logical columns 4*p .. 4*p+3 of both column blocks, p = piece ^ (row & 7).
    const int lp = (t & 7) ^ (c & 7);
    float4 *DM = reinterpret_cast<float4 *>(dstates_m + base) + c * 8 + ((((lp >> 1) ^ (c & 3)) << 1) | (lp & 1));
    const float *gm = gamma + (size_t)blockIdx.y * N * 64 + c;
    float *cr = carry + (size_t)blockIdx.y * N * 64 + c;
    float4 r0 = make_float4(0.f, 0.f, 0.f, 0.f), r1 = r0;
    // this thread's logical columns 4*lp .. 4*lp+3 and 32 + 4*lp .. of row c in a row-major state
    const size_t io = ((size_t)blockIdx.y * 64 + c) * 64 + 4 * lp;
    if (s_in != nullptr) {
        r0 = *reinterpret_cast<const float4 *>(s_in + io);
        r1 = *reinterpret_cast<const float4 *>(s_in + io + 32);
    }
    for (int i = 0; i < N; i += kAhead) {
        float4 u0[kAhead], u1[kAhead];
        float g[kAhead];
#pragma unroll
        for (int j = 0; j < kAhead; ++j)
            if (i + j < N) {
                u0[j] = S[(size_t)(i + j) * 1024];
                u1[j] = S[(size_t)(i + j) * 1024 + 512];
                g[j] = gm[(size_t)(i + j) * 64];
            }
#pragma unroll
        for (int j = 0; j < kAhead; ++j)
            if (i + j < N) {
                S[(size_t)(i + j) * 1024] = round4_tf32(r0);
                S[(size_t)(i + j) * 1024 + 512] = round4_tf32(r1);
                r0 = fma4(g[j], r0, u0[j]);
                r1 = fma4(g[j], r1, u1[j]);
            }
    }
    float4 d0 = make_float4(0.f, 0.f, 0.f, 0.f), d1 = d0;
    if (ds_out != nullptr) {
        d0 = *reinterpret_cast<const float4 *>(ds_out + io);
        d1 = *reinterpret_cast<const float4 *>(ds_out + io + 32);
    }
    for (int i = N - 1; i >= 0; i -= kBack) {
        float4 w0[kBack], w1[kBack], s0[kBack], s1[kBack];
        float g[kBack];
#pragma unroll
        for (int j = 0; j < kBack; ++j) {
            const int ch = i - j;
            if (ch >= 0) {
                w0[j] = D[(size_t)ch * 1024];
                w1[j] = D[(size_t)ch * 1024 + 512];
                g[j] = gm[(size_t)ch * 64];
                if (ch + 1 < N) {
                    s0[j] = S[(size_t)(ch + 1) * 1024];
                    s1[j] = S[(size_t)(ch + 1) * 1024 + 512];
                } else {              // the last chunk leaves the final state, still in registers
                    s0[j] = r0;
                    s1[j] = r1;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kBack; ++j) {
            const int ch = i - j;
            if (ch >= 0) {            // uniform over the block
                float dot = s0[j].x * d0.x + s0[j].y * d0.y + s0[j].z * d0.z + s0[j].w * d0.w +
                            s1[j].x * d1.x + s1[j].y * d1.y + s1[j].z * d1.z + s1[j].w * d1.w;
                const float4 e0 = round4_tf32(make_float4(g[j] * d0.x, g[j] * d0.y, g[j] * d0.z, g[j] * d0.w));
                const float4 e1 = round4_tf32(make_float4(g[j] * d1.x, g[j] * d1.y, g[j] * d1.z, g[j] * d1.w));
                D[(size_t)ch * 1024] = e0;
                D[(size_t)ch * 1024 + 512] = e1;
                DM[(size_t)ch * 1024] = e0;
                DM[(size_t)ch * 1024 + 512] = e1;
                d0 = fma4(g[j], d0, w0[j]);
                d1 = fma4(g[j], d1, w1[j]);
                dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                if ((t & 7) == 0) cr[(size_t)ch * 64] = dot;
            }
        }
    }
    if (ds_in != nullptr) {
        *reinterpret_cast<float4 *>(ds_in + io) = d0;
        *reinterpret_cast<float4 *>(ds_in + io + 32) = d1;
    }
}

// The same two scans for calls with few sequences: one warp per row, lane l holds logical columns l
// and 32 + l (the same offset in the two column blocks, so a warp touches one 128-byte line per
// block), 32 chunks of loads in flight.  Four times the threads and twice the look-ahead of the kernel
// above; slower than it when there are enough sequences to fill the GPU.
constexpr int kTileRows = 4, kLook1 = 32;
__global__ void __launch_bounds__(32 * kTileRows)
state_scan_bwd_tiles1(float *__restrict__ states, float *__restrict__ dstates, float *__restrict__ dstates_m,
                      const float *__restrict__ gamma, float *__restrict__ carry, const float *__restrict__ s_in,
                      const float *__restrict__ ds_out, float *__restrict__ ds_in, int N)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const int lane = threadIdx.x & 31, c = kTileRows * blockIdx.x + (threadIdx.x >> 5);
    const size_t base = (size_t)blockIdx.y * N * 4096;
    const int offk = c * 32 + ((((lane >> 2) ^ (c & 7)) << 2) | (lane & 3));
    const int offm = c * 32 + ((((lane >> 3) ^ (c & 3)) << 3) | (lane & 7));
    float *S = states + base + offk;
    float *D = dstates + base + offk;
    float *DM = dstates_m + base + offm;
    const float *gm = gamma + (size_t)blockIdx.y * N * 64 + c;
    float *cr = carry + (size_t)blockIdx.y * N * 64 + c;
    const size_t io = ((size_t)blockIdx.y * 64 + c) * 64 + lane;       // row-major state: columns lane, lane + 32
    float r0 = 0.f, r1 = 0.f;
    if (s_in != nullptr) {
        r0 = s_in[io];
        r1 = s_in[io + 32];
    }
    for (int i = 0; i < N; i += kLook1) {
        float u0[kLook1], u1[kLook1], g[kLook1];
        const float *ps = S + (size_t)i * 4096;
        const float *pg = gm + (size_t)i * 64;
#pragma unroll
        for (int j = 0; j < kLook1; ++j) {
            if (i + j < N) {
                u0[j] = ps[0];
                u1[j] = ps[2048];
                g[j] = *pg;
            }
            ps += 4096;
            pg += 64;
        }
        float *pw = S + (size_t)i * 4096;
#pragma unroll
        for (int j = 0; j < kLook1; ++j) {
            if (i + j < N) {
                pw[0] = round_tf32(r0);
                pw[2048] = round_tf32(r1);
                r0 = fmaf(g[j], r0, u0[j]);
                r1 = fmaf(g[j], r1, u1[j]);
            }
            pw += 4096;
        }
    }
    float d0 = 0.f, d1 = 0.f;
    if (ds_out != nullptr) {
        d0 = ds_out[io];
        d1 = ds_out[io + 32];
    }
    constexpr int kB = kLook1 / 2;
    for (int i = N - 1; i >= 0; i -= kB) {
        float w0[kB], w1[kB], s0[kB], s1[kB], g[kB];
#pragma unroll
        for (int j = 0; j < kB; ++j) {
            const int ch = i - j;
            if (ch >= 0) {
                w0[j] = D[(size_t)ch * 4096];
                w1[j] = D[(size_t)ch * 4096 + 2048];
                g[j] = gm[(size_t)ch * 64];
                if (ch + 1 < N) {
                    s0[j] = S[(size_t)(ch + 1) * 4096];
                    s1[j] = S[(size_t)(ch + 1) * 4096 + 2048];
                } else {              // the last chunk leaves the final state, still in registers
                    s0[j] = r0;
                    s1[j] = r1;
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kB; ++j) {
            const int ch = i - j;
            if (ch >= 0) {            // uniform over the block
                float dot = fmaf(s0[j], d0, s1[j] * d1);
                const float e0 = round_tf32(g[j] * d0), e1 = round_tf32(g[j] * d1);
                D[(size_t)ch * 4096] = e0;
                D[(size_t)ch * 4096 + 2048] = e1;
                DM[(size_t)ch * 4096] = e0;
                DM[(size_t)ch * 4096 + 2048] = e1;
                d0 = fmaf(g[j], d0, w0[j]);
                d1 = fmaf(g[j], d1, w1[j]);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
                if (lane == 0) cr[(size_t)ch * 64] = dot;
            }
        }
    }
    if (ds_in != nullptr) {
        ds_in[io] = d0;
        ds_in[io + 32] = d1;
    }
}

// ---- the same scans with the value-channel gate (full gate G = alpha^T beta of Eq. gate_gla) ---------
// The state decays along its rows by gamma (key channels) and along its columns by gamma_v (value
// channels): S_[i+1] = diag(gamma_i) S_[i] diag(gamma_v_i) + U_i, and the mirror image for D.  Row-major
// states only (warp-MMA family); stored states and diag(gamma) D diag(gamma_v) are rounded to tf32.
__global__ void __launch_bounds__(kScanThreads)
state_scan_fwd_beta(float *__restrict__ states, const float *__restrict__ gamma, const float *__restrict__ gamma_v,
                    float *__restrict__ s_final, int N, int dk, int dv)
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
                st[(size_t)(i + j) * sstride] = round4_tf32(run);
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
                    const float *__restrict__ gamma_v, float *__restrict__ carry, int N, int dk, int dv)
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
                if (e < dv) D[(size_t)ch * sstride + e] = round_tf32(g[j][r] * run[r]);
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

dig_status launch_state_scan_fwd(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio, bool tiles, bool tf32)
{
    const dim3 grid((g.dk * g.dv / 4 + kScanThreads - 1) / kScanThreads, g.B * g.H);
    if (tiles && (g.dk != 64 || g.dv != 64)) return DIG_ERR_UNSUPPORTED;
    // the state after the last chunk goes to the caller if asked for, else to the workspace block the
    // backward scan reads it from (null in a forward-only workspace)
    float *fin = sio.s_out != nullptr ? sio.s_out : w.sfinal;
    KernelTimer t(KID_SCAN_FWD, s);
    if ((long long)grid.x * grid.y * kScanThreads < 16384) {       // few sequences: one element per thread
        const dim3 grid1((g.dk * g.dv + kScan1Threads - 1) / kScan1Threads, g.B * g.H);
        if (tiles)
            launch_pdl(state_scan_fwd1<true, true>, grid1, dim3(kScan1Threads), 0, s, w.states, (const float *)w.gamma, sio.s_in,
                       fin, g.N, g.dk, g.dv);
        else if (tf32)
            state_scan_fwd1<false, true><<<grid1, kScan1Threads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
        else
            state_scan_fwd1<false, false><<<grid1, kScan1Threads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
        return cuda_ok(cudaGetLastError());
    }
    if (tiles)
        launch_pdl(state_scan_fwd<true>, grid, dim3(kScanThreads), 0, s, w.states, (const float *)w.gamma, sio.s_in, fin, g.N,
                   g.dk, g.dv);
    else if (tf32)
        state_scan_fwd<false, true><<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, sio.s_in, fin, g.N, g.dk, g.dv);
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

dig_status launch_state_scan_bwd_tiles(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio)
{
    if (g.dk != 64 || g.dv != 64) return DIG_ERR_UNSUPPORTED;
    KernelTimer t(KID_SCAN_BWD, s);
    if (g.B * g.H < 16)      // few sequences: the finer kernel with the deeper look-ahead
        launch_pdl(state_scan_bwd_tiles1, dim3(64 / kTileRows, g.B * g.H), dim3(32 * kTileRows), 0, s, w.states, w.dstates,
                   w.dstates_m, (const float *)w.gamma, w.carry, sio.s_in, sio.ds_out, sio.ds_in, g.N);
    else
        launch_pdl(state_scan_bwd_tiles, dim3(8, g.B * g.H), dim3(64), 0, s, w.states, w.dstates, w.dstates_m,
                   (const float *)w.gamma, w.carry, sio.s_in, sio.ds_out, sio.ds_in, g.N);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_state_scan_fwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s)
{
    const dim3 grid((g.dk * g.dv / 4 + kScanThreads - 1) / kScanThreads, g.B * g.H);
    KernelTimer t(KID_SCAN_FWD, s);
    state_scan_fwd_beta<<<grid, kScanThreads, 0, s>>>(w.states, w.gamma, gamma_v, w.sfinal, g.N, g.dk, g.dv);
    return cuda_ok(cudaGetLastError());
}

dig_status launch_state_scan_bwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s)
{
    const dim3 grid((g.dk + kRowsPerBlock - 1) / kRowsPerBlock, g.B * g.H);
    KernelTimer t(KID_SCAN_BWD, s);
    state_scan_bwd_beta<<<grid, 32 * kRowsPerBlock, 0, s>>>(w.states, w.dstates, w.gamma, gamma_v, w.carry, g.N, g.dk, g.dv);
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
