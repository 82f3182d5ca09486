// Gate transform of the key-channel decay (Eq. gate_gla): alpha = sigmoid(x)^(1/tau), produced
// directly as log(alpha) = logsigmoid(x)/tau, which is what the chunkwise operator consumes.
// Elementwise and bandwidth-bound: 16-byte loads, 8 elements per thread.
#include "dig_common.cuh"

namespace dig {
namespace {

constexpr int kMaxHeads = 256;
struct InvTau { float v[kMaxHeads]; };

__device__ __forceinline__ float log_sigmoid(float x)
{
    // log(1/(1+e^-x)) = min(x, 0) - log1p(e^-|x|), without overflow on either side.  e^-|x| <= 1 comes
    // from the fast exponential (a few ulp; its error enters the result damped by 1/(1+t)), the
    // logarithm stays the accurate one: the result keeps an absolute error near 1e-7.
    return fminf(x, 0.f) - log1pf(__expf(-fabsf(x)));
}

template <typename T>
__global__ void __launch_bounds__(256)
gate_logsigmoid(const T *__restrict__ g, float *__restrict__ gate, size_t n8, int H, int dk,
                InvTau inv_tau)
{
    pdl_wait();
    pdl_launch_dependents();      // only once this kernel's own predecessor has completed
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += stride) {
        const size_t e = i * 8;
        const int h = (int)((e / dk) % H);
        const float it = inv_tau.v[h];
        const float4 a = load4(g + e), b = load4(g + e + 4);
        store4(gate + e, make_float4(log_sigmoid(a.x) * it, log_sigmoid(a.y) * it,
                                     log_sigmoid(a.z) * it, log_sigmoid(a.w) * it));
        store4(gate + e + 4, make_float4(log_sigmoid(b.x) * it, log_sigmoid(b.y) * it,
                                         log_sigmoid(b.z) * it, log_sigmoid(b.w) * it));
    }
}

}  // namespace

dig_status launch_gate(const void *g, const float *tau_host, float *gate, int B, int L, int H,
                       int dk, int dtype, cudaStream_t stream)
{
    if (H > kMaxHeads) return DIG_ERR_UNSUPPORTED;
    InvTau it;
    for (int h = 0; h < H; ++h) {
        if (!(tau_host[h] > 0.f)) return DIG_ERR_INVALID_ARG;
        it.v[h] = 1.0f / tau_host[h];
    }
    const size_t n8 = (size_t)B * L * H * dk / 8;
    const int blocks = (int)((n8 + 255) / 256 < 148 * 16 ? (n8 + 255) / 256 : 148 * 16);
    KernelTimer t(KID_GATE, stream);
    if (dtype == DIG_F32)
        launch_pdl(gate_logsigmoid<float>, dim3(blocks), dim3(256), 0, stream, (const float *)g, gate, n8, H, dk, it);
    else
        launch_pdl(gate_logsigmoid<__nv_bfloat16>, dim3(blocks), dim3(256), 0, stream, (const __nv_bfloat16 *)g, gate, n8, H, dk, it);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
