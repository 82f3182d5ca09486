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
    // log(1/(1+e^-x)) = min(x, 0) - log1p(t), t = e^-|x| in (0, 1], without overflow on either side.
    // t: 2^(-|x| log2 e) with the rounding error of the product carried along (the fast exponential
    // alone would lose |x| * 6e-8 of relative accuracy for large |x|).
    // log1p(t) = t (1 + t r(t)), r a degree-8 polynomial fitted at Chebyshev nodes of [0, 1]: relative
    // error 1.5e-7 in fp32 over the whole interval, and exact behaviour t - t^2/2 as t -> 0, so small
    // results (large positive x) keep their relative accuracy.
    const float ax = -fabsf(x);
    const float hi = ax * 1.44269502162933349609375f;
    const float lo = fmaf(ax, 1.44269502162933349609375f, -hi) + ax * 1.925963033500011e-8f;
    float t;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(hi));
    t = fmaf(t, lo * 0.693147182464599609375f, t);
    float r = -4.466211586e-03f;
    r = fmaf(r, t, 2.522405428e-02f);
    r = fmaf(r, t, -6.675772493e-02f);
    r = fmaf(r, t, 1.156184543e-01f);
    r = fmaf(r, t, -1.584756571e-01f);
    r = fmaf(r, t, 1.985410623e-01f);
    r = fmaf(r, t, -2.498652617e-01f);
    r = fmaf(r, t, 3.333284189e-01f);
    r = fmaf(r, t, -4.999999698e-01f);
    return fminf(x, 0.f) - t * fmaf(t, r, 1.f);
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
    const int sms = device_sm_count();
    if (sms <= 0) return DIG_ERR_CUDA;
    const int blocks = (int)((n8 + 255) / 256 < (size_t)sms * 16 ? (n8 + 255) / 256 : (size_t)sms * 16);
    KernelTimer t(KID_GATE, stream);
    if (dtype == DIG_F32)
        launch_pdl(gate_logsigmoid<float>, dim3(blocks), dim3(256), 0, stream, (const float *)g, gate, n8, H, dk, it);
    else
        launch_pdl(gate_logsigmoid<__nv_bfloat16>, dim3(blocks), dim3(256), 0, stream, (const __nv_bfloat16 *)g, gate, n8, H, dk, it);
    return cuda_ok(cudaGetLastError());
}

}  // namespace dig
