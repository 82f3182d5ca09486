// Shared device/host helpers of the DiG GLA library: problem descriptor, scan-order index map,
// storage-type conversion.  Internal; the public surface is include/dig_gla.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dig_gla.h"

namespace dig {

// Geometry of one GLA call, passed by value to every kernel.
struct Geom {
    int B, H, gh, gw, L, dk, dv, C, N, dir;   // N = ceil(L / C) chunks per (batch, head)
};

// Canonical token (y*gw + x) visited at scan position p.  Row orders walk the row-major
// sequence forwards / backwards; column orders walk the transposed token matrix
// (Algorithm 1: "flip" and "transpose" of the reshaped token matrix).
__host__ __device__ __forceinline__ int scan_token(int p, int dir, int gh, int gw, int L)
{
    if (dir & 1) p = L - 1 - p;
    if (dir & 2) {
        const int x = p / gh, y = p - x * gh;
        return y * gw + x;
    }
    return p;
}

// Element offset of token t, head h in a [B][L][H][d] tensor.
__host__ __device__ __forceinline__ size_t tok_offset(const Geom &g, int b, int t, int h, int d)
{
    return (((size_t)b * g.L + t) * g.H + h) * (size_t)d;
}

// ---- storage conversion ---------------------------------------------------------------
// Load 4 consecutive elements (16-byte aligned for float, 8-byte for bf16) as floats.
__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p)
{
    const uint2 u = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162 *>(&u.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162 *>(&u.y);
    return make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
}
__device__ __forceinline__ void store4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 v)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
    __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t *>(&a);
    u.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = u;
}

// ---- launch plumbing shared by the .cu files --------------------------------------------
// Optional state arguments of the recurrence (all [B][H][d_k][d_v] fp32 row-major, any may be null):
// the state before the first scan position, the state after the last one, the gradient with
// respect to that final state, and the gradient with respect to the start state.
struct StateIO {
    const float *s_in;
    float *s_out;
    const float *ds_out;
    float *ds_in;
};

// Arguments of the variant with the value-channel gate (all null otherwise): log(beta) [B][L][H][d_v]
// and the gradient with respect to it.
struct BetaIO {
    const float *bgate;
    float *dbgate;
};

struct GlaArgs {
    StateIO sio;
    BetaIO bio;
    const void *q, *k, *v;
    const float *gate;
    void *out;                   // forward
    const void *d_out;           // backward
    void *dq, *dk, *dv;
    float *dgate;
    float *ws;                   // workspace base (fp32 view)
    Geom g;
    int dtype;
    int accumulate;              // outputs are added to what the (fp32) output buffers hold
    cudaStream_t stream;
};

// Workspace carving (all fp32, every block 256-byte aligned).
//   states  [B*H][N][dk][dv]   chunk-local K^T V, turned in place into the state entering each chunk
//   gamma   [B*H][N][dk]       exp(sum of the chunk's gates)
//   dstates [B*H][N][dk][dv]   (backward) chunk-local Q^T dO, turned in place into dL/d(state leaving the chunk)
//   carry   [B*H][N][dk]       (backward) gate-gradient carried in from later chunks
struct Workspace {
    float *states, *gamma, *dstates, *carry, *sfinal;
    size_t bytes;
};
inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }
inline Workspace carve_workspace(float *base, const Geom &g, bool backward)
{
    Workspace w{};
    const size_t bh = (size_t)g.B * g.H;
    const size_t st = align256(bh * g.N * g.dk * g.dv * sizeof(float));
    const size_t gm = align256(bh * g.N * g.dk * sizeof(float));
    char *p = reinterpret_cast<char *>(base);
    w.states = reinterpret_cast<float *>(p);            p += st;
    w.gamma = reinterpret_cast<float *>(p);             p += gm;
    w.bytes = st + gm;
    if (backward) {
        w.dstates = reinterpret_cast<float *>(p);       p += st;
        w.carry = reinterpret_cast<float *>(p);         p += gm;
        const size_t fin = align256(bh * g.dk * g.dv * sizeof(float));
        w.sfinal = reinterpret_cast<float *>(p);        p += fin;
        w.bytes += st + gm + fin;
    }
    return w;
}

// Kernel families (each returns a dig_status).
dig_status fma_gla_fwd(const GlaArgs &a);
dig_status fma_gla_bwd(const GlaArgs &a);
bool fma_supports(int dk, int dv, int chunk, int dtype, bool backward);
dig_status mma_gla_fwd(const GlaArgs &a);
dig_status mma_gla_bwd(const GlaArgs &a);
bool mma_supports(int dk, int dv, int chunk, int dtype, bool backward, bool beta = false);
size_t mma_beta_workspace_bytes(const Geom &g, bool backward);

// Chunk-state scans, shared by both families (plain fp32 FMA, bandwidth-bound).
dig_status launch_state_scan_fwd(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio, bool tf32 = false);
dig_status launch_state_scan_bwd(const Workspace &w, const Geom &g, cudaStream_t s, const StateIO &sio, bool tf32 = false);
// Scans with the value-channel gate (row-major states, tf32-rounded results) and the cross-chunk part of its gradient.
dig_status launch_state_scan_fwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s, bool tf32);
dig_status launch_state_scan_bwd_beta(const Workspace &w, const float *gamma_v, const Geom &g, cudaStream_t s, bool tf32);
dig_status launch_beta_carry(float *dbgate, float *xtot, const Geom &g, cudaStream_t s);

// Device status word (bounded waits report here).
int *device_status_ptr();
// Streaming multiprocessors of the current device (cached per device), 0 on error.
int device_sm_count();
// Raises a kernel's dynamic shared memory limit to at least `bytes`; the driver is asked only when the
// value grows (remembered per kernel and device).
dig_status ensure_dynamic_smem(const void *kernel, size_t bytes);

// Optional per-kernel timing (dig_profile_*): when enabled, every launch site brackets its
// kernel with two CUDA events on the launching stream.
enum KernelId {
    KID_GATE = 0, KID_DWCONV, KID_DWCONV_WGRAD, KID_OUTGATE, KID_SCAN_FWD, KID_SCAN_BWD,
    KID_FMA_STATE, KID_FMA_OUT, KID_FMA_BWD,
    KID_MMA_STATE, KID_MMA_OUT, KID_MMA_BWD,
    KID_SW_LOCAL, KID_SW_SCAN, KID_SW_FWD, KID_SW_BWD,
    KID_COUNT
};
struct KernelTimer {
    KernelTimer(int kernel_id, cudaStream_t stream);
    ~KernelTimer();
    int slot;
    cudaStream_t stream;
};

// ---- programmatic dependent launch -------------------------------------------------------
// Kernels launched through launch_pdl may be scheduled while the previous kernel of the stream is
// still draining; they call pdl_wait() before their first access to global memory, which blocks
// until that kernel has completed and its writes are visible.  pdl_launch_dependents() lets the
// next kernel of the stream do the same with respect to this one; it is called after pdl_wait(), so
// that early launches cannot cascade past a kernel whose own predecessor is still running.  Both are no-ops for a kernel
// launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline dig_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? DIG_OK : DIG_ERR_CUDA; }

}  // namespace dig
