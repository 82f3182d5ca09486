// extern "C" entry points: argument validation, kernel-family choice, launches.
#include <atomic>
#include <cstring>
#include <map>
#include <mutex>
#include <utility>
#include <vector>

#include "dig_common.cuh"
#include "sweep.cuh"
#include "umma.cuh"

namespace dig {

dig_status launch_gate(const void *g, const float *tau_host, float *gate, int B, int L, int H,
                       int dk, int dtype, cudaStream_t stream);
dig_status launch_dwconv(const void *x, const void *w, const void *bias, void *y, int B, int gh,
                         int gw, int D, int dir, int dtype, cudaStream_t stream);
size_t outgate_bwd_workspace_bytes(long long rows, int dv);
dig_status launch_outgate_fwd_mixed(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                                    long long rows, int dv, float eps, int dtype, cudaStream_t stream);
dig_status launch_outgate_fwd(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                              long long rows, int dv, float eps, int dtype, cudaStream_t stream);
dig_status launch_outgate_bwd(const void *o, const void *r, const void *dz, const float *ln_w, const float *ln_b,
                              void *d_o, void *d_r, float *dln_w, float *dln_b, long long rows, int dv, float eps,
                              int dtype, float *partial, cudaStream_t stream);
size_t dwconv_bwd_workspace_bytes(int B, int gh, int gw, int D);
dig_status launch_dwconv_bwd(const void *x, const void *w, const void *dy, void *dx, float *dw, float *dbias,
                             int B, int gh, int gw, int D, int dir, int dtype, float *partial, cudaStream_t stream);

namespace {

std::atomic<int> g_impl{DIG_IMPL_AUTO};

// Written by device code when a bounded wait expires; read and cleared by dig_last_device_status.
__device__ int g_device_status = 0;

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool valid_dtype(int d) { return d == DIG_F32 || d == DIG_BF16 || d == DIG_BF16_F32OUT; }
bool valid_chunk(int c) { return c == 16 || c == 32 || c == 64 || c == 128; }
bool valid_dim(int d) { return d >= 8 && d <= 128 && (d % 8) == 0; }

bool valid_geometry(int B, int H, int gh, int gw, int dk, int dv, int chunk, int dir, int dtype)
{
    if (B <= 0 || H <= 0 || gh <= 0 || gw <= 0) return false;
    if ((long long)gh * gw > (1ll << 24)) return false;
    if ((long long)B * H > 65535) return false;
    return valid_dim(dk) && valid_dim(dv) && valid_chunk(chunk) && dir >= 0 && dir <= 3 &&
           valid_dtype(dtype);
}

Geom make_geom(int B, int H, int gh, int gw, int dk, int dv, int chunk, int dir)
{
    Geom g;
    g.B = B; g.H = H; g.gh = gh; g.gw = gw; g.L = gh * gw; g.dk = dk; g.dv = dv; g.C = chunk;
    g.N = (g.L + chunk - 1) / chunk; g.dir = dir;
    return g;
}

// DIG_IMPL_FMA / DIG_IMPL_TENSOR / DIG_IMPL_MMA, or a negative status.
// The tcgen05 kernels take the requested chunk size as it is (they work in 64-token tiles and treat
// shorter chunks as sub-chunks of a tile, longer ones as 64).
int tile_chunk(int impl, int chunk) { (void)impl; return chunk; }

int choose_impl(int dk, int dv, int chunk, int dtype, bool backward)
{
    const int want = g_impl.load();
    const bool t_ok = sweep_supports(dk, dv, chunk, dtype);
    const bool f_ok = fma_supports(dk, dv, chunk, dtype, backward);
    const bool m_ok = mma_supports(dk, dv, chunk, dtype, backward);
    if (want == DIG_IMPL_TENSOR) return t_ok ? DIG_IMPL_TENSOR : -(int)DIG_ERR_UNSUPPORTED;
    if (want == DIG_IMPL_FMA) return f_ok ? DIG_IMPL_FMA : -(int)DIG_ERR_UNSUPPORTED;
    if (want == DIG_IMPL_MMA) return m_ok ? DIG_IMPL_MMA : -(int)DIG_ERR_UNSUPPORTED;
    if (t_ok) return DIG_IMPL_TENSOR;
    if (m_ok) return DIG_IMPL_MMA;
    if (f_ok) return DIG_IMPL_FMA;
    return -(int)DIG_ERR_UNSUPPORTED;
}

}  // namespace

// ---- per-kernel timing ---------------------------------------------------------------------
namespace {
constexpr int kMaxTimed = 32768;
const char *const kKernelNames[KID_COUNT] = {
    "gate_logsigmoid", "srem_dwconv3x3", "srem_dwconv_wgrad", "gla_outgate", "state_scan_fwd", "state_scan_bwd",
    "fma_chunk_state", "fma_chunk_out", "fma_chunk_bwd",
    "mma_chunk_state", "mma_chunk_out", "mma_chunk_bwd",
    "sweep_local", "seg_scan", "sweep_fwd", "sweep_bwd"};
struct Profile {
    bool on = false;
    std::vector<cudaEvent_t> ev;      // 2 per timed launch, created lazily and reused
    std::vector<int> kernel_of;       // kernel id of each recorded pair
    int launches[KID_COUNT] = {};
};
Profile g_prof;
}  // namespace

KernelTimer::KernelTimer(int kernel_id, cudaStream_t s) : slot(-1), stream(s)
{
    if (!g_prof.on) return;
    g_prof.launches[kernel_id]++;
    const int n = (int)g_prof.kernel_of.size();
    if (n >= kMaxTimed) return;
    while ((int)g_prof.ev.size() < 2 * (n + 1)) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        g_prof.ev.push_back(e);
    }
    g_prof.kernel_of.push_back(kernel_id);
    slot = n;
    cudaEventRecord(g_prof.ev[2 * slot], stream);
}
KernelTimer::~KernelTimer()
{
    if (slot >= 0) cudaEventRecord(g_prof.ev[2 * slot + 1], stream);
}

// One CTA waits on an mbarrier that nothing ever arrives on, with a short limit: exercises the path a
// bounded wait takes when it gives up (status word, normal return).
__global__ void wait_that_expires(int *status, unsigned long long limit_ns)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        umma::mbar_init(&bar, 1);
        umma::fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) umma::mbar_wait(&bar, 0, status, limit_ns);
}

int *device_status_ptr()
{
    int *p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_device_status) != cudaSuccess) return nullptr;
    return p;
}

int device_sm_count()
{
    static std::atomic<int> cached[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    int n = cached[dev].load();
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev].store(n);
    }
    return n;
}

dig_status ensure_dynamic_smem(const void *kernel, size_t bytes)
{
    static std::mutex mu;
    static std::map<std::pair<const void *, int>, size_t> granted;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIG_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    size_t &have = granted[std::make_pair(kernel, dev)];
    if (bytes <= have) return DIG_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return DIG_ERR_CUDA;
    have = bytes;
    return DIG_OK;
}

}  // namespace dig

using namespace dig;

extern "C" {

dig_status dig_set_impl(int impl)
{
    if (impl < DIG_IMPL_AUTO || impl > DIG_IMPL_MMA) return DIG_ERR_INVALID_ARG;
    g_impl.store(impl);
    return DIG_OK;
}

int dig_gla_query_impl(int d_k, int d_v, int chunk, int dtype, int backward)
{
    if (!valid_dim(d_k) || !valid_dim(d_v) || !valid_chunk(chunk) || !valid_dtype(dtype))
        return -(int)DIG_ERR_INVALID_ARG;
    return choose_impl(d_k, d_v, chunk, dtype, backward != 0);
}

size_t dig_gla_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                               int dtype, int backward)
{
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, 0, dtype)) return 0;
    // sized for whichever family may serve the call
    const Geom g = make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, 0);
    size_t need = 0;
    if (sweep_supports(d_k, d_v, chunk, dtype)) need = sweep_workspace_bytes(g, backward != 0);
    if (fma_supports(d_k, d_v, chunk, dtype, backward != 0) || mma_supports(d_k, d_v, chunk, dtype, backward != 0)) {
        const size_t other = carve_workspace(nullptr, g, backward != 0).bytes;
        need = other > need ? other : need;
    }
    return need;
}

dig_status dig_gate_logsigmoid(const void *g, const float *tau_per_head, float *gate, int B, int L,
                               int H, int d_k, int dtype, void *cuda_stream)
{
    if (!g || !tau_per_head || !gate || !aligned16(g) || !aligned16(gate)) return DIG_ERR_INVALID_ARG;
    if (B <= 0 || L <= 0 || H <= 0 || !valid_dim(d_k) || !valid_dtype(dtype)) return DIG_ERR_INVALID_ARG;
    return launch_gate(g, tau_per_head, gate, B, L, H, d_k, dtype, (cudaStream_t)cuda_stream);
}

dig_status dig_gla_fwd_state(const void *q, const void *k, const void *v, const float *gate, const float *s_in,
                             void *out, float *s_out,
                       int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk,
                       int direction, int dtype, void *workspace, size_t workspace_bytes,
                       void *cuda_stream)
{
    if (!q || !k || !v || !gate || !out) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(out))
        return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype)) return DIG_ERR_INVALID_ARG;
    const size_t need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 0);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    const int impl = choose_impl(d_k, d_v, chunk, dtype, false);
    if (impl < 0) return (dig_status)(-impl);
    if ((s_in && !aligned16(s_in)) || (s_out && !aligned16(s_out))) return DIG_ERR_INVALID_ARG;
    GlaArgs a{};
    a.sio.s_in = s_in; a.sio.s_out = s_out;
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.out = out;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, tile_chunk(impl, chunk), direction);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return impl == DIG_IMPL_TENSOR ? sweep_gla_fwd(a) : impl == DIG_IMPL_MMA ? mma_gla_fwd(a) : fma_gla_fwd(a);
}

dig_status dig_gla_bwd_state(const void *q, const void *k, const void *v, const float *gate,
                             const void *d_out, const float *s_in, const float *ds_out, void *dq, void *dk, void *dv,
                             float *dgate, float *ds_in, int B, int H,
                       int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                       void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !d_out || !dq || !dk || !dv || !dgate) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(d_out) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(dgate))
        return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype)) return DIG_ERR_INVALID_ARG;
    const size_t need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 1);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    const int impl = choose_impl(d_k, d_v, chunk, dtype, true);
    if (impl < 0) return (dig_status)(-impl);
    if ((s_in && !aligned16(s_in)) || (ds_out && !aligned16(ds_out)) || (ds_in && !aligned16(ds_in))) return DIG_ERR_INVALID_ARG;
    GlaArgs a{};
    a.sio.s_in = s_in; a.sio.ds_out = ds_out; a.sio.ds_in = ds_in;
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.d_out = d_out;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dgate = dgate;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, tile_chunk(impl, chunk), direction);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return impl == DIG_IMPL_TENSOR ? sweep_gla_bwd(a) : impl == DIG_IMPL_MMA ? mma_gla_bwd(a) : fma_gla_bwd(a);
}

dig_status dig_gla_fwd(const void *q, const void *k, const void *v, const float *gate, void *out,
                       int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction,
                       int dtype, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return dig_gla_fwd_state(q, k, v, gate, nullptr, out, nullptr, B, H, grid_h, grid_w, d_k, d_v, chunk, direction,
                             dtype, workspace, workspace_bytes, cuda_stream);
}

dig_status dig_gla_bwd(const void *q, const void *k, const void *v, const float *gate,
                       const void *d_out, void *dq, void *dk, void *dv, float *dgate, int B, int H,
                       int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                       void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return dig_gla_bwd_state(q, k, v, gate, d_out, nullptr, nullptr, dq, dk, dv, dgate, nullptr, B, H, grid_h, grid_w,
                             d_k, d_v, chunk, direction, dtype, workspace, workspace_bytes, cuda_stream);
}

dig_status dig_srem_dwconv(const void *x, const void *w, const void *bias, void *y, int B,
                           int grid_h, int grid_w, int D, int direction, int dtype, void *cuda_stream)
{
    if (!x || !w || !y || !aligned16(x) || !aligned16(w) || !aligned16(y)) return DIG_ERR_INVALID_ARG;
    if (bias && !aligned16(bias)) return DIG_ERR_INVALID_ARG;
    if (B <= 0 || grid_h <= 0 || grid_w <= 0 || D <= 0 || (D % 8) != 0) return DIG_ERR_INVALID_ARG;
    if (direction < 0 || direction > 3 || !valid_dtype(dtype)) return DIG_ERR_INVALID_ARG;
    return launch_dwconv(x, w, bias, y, B, grid_h, grid_w, D, direction, dtype, (cudaStream_t)cuda_stream);
}

size_t dig_srem_dwconv_bwd_workspace_bytes(int B, int grid_h, int grid_w, int D)
{
    if (B <= 0 || grid_h <= 0 || grid_w <= 0 || D <= 0 || (D % 8) != 0) return 0;
    if ((long long)B * grid_h * grid_w > (1ll << 30)) return 0;
    return dwconv_bwd_workspace_bytes(B, grid_h, grid_w, D);
}

dig_status dig_srem_dwconv_bwd(const void *x, const void *w, const void *dy, void *dx, float *dw, float *dbias,
                               int B, int grid_h, int grid_w, int D, int direction, int dtype, void *workspace,
                               size_t workspace_bytes, void *cuda_stream)
{
    if (!x || !w || !dy || !dx || !dw) return DIG_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w) || !aligned16(dy) || !aligned16(dx) || !aligned16(dw)) return DIG_ERR_INVALID_ARG;
    if (dbias && !aligned16(dbias)) return DIG_ERR_INVALID_ARG;
    if (direction < 0 || direction > 3 || !valid_dtype(dtype)) return DIG_ERR_INVALID_ARG;
    const size_t need = dig_srem_dwconv_bwd_workspace_bytes(B, grid_h, grid_w, D);
    if (need == 0) return DIG_ERR_INVALID_ARG;
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    return launch_dwconv_bwd(x, w, dy, dx, dw, dbias, B, grid_h, grid_w, D, direction, dtype,
                             reinterpret_cast<float *>(workspace), (cudaStream_t)cuda_stream);
}

static bool outgate_sizes_ok(long long rows, int d_v, float eps)
{
    return rows > 0 && rows <= (1ll << 40) && d_v > 0 && d_v <= 128 && (d_v % 8) == 0 && eps >= 0.f;
}

dig_status dig_gla_outgate_fwd(const void *o, const void *r, const float *ln_w, const float *ln_b, void *z,
                               long long rows, int d_v, float eps, int dtype, void *cuda_stream)
{
    if (!o || !r || !z || !aligned16(o) || !aligned16(r) || !aligned16(z)) return DIG_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || !outgate_sizes_ok(rows, d_v, eps)) return DIG_ERR_INVALID_ARG;
    return launch_outgate_fwd(o, r, ln_w, ln_b, z, rows, d_v, eps, dtype, (cudaStream_t)cuda_stream);
}

size_t dig_gla_outgate_bwd_workspace_bytes(long long rows, int d_v)
{
    if (!outgate_sizes_ok(rows, d_v, 0.f)) return 0;
    return outgate_bwd_workspace_bytes(rows, d_v);
}

dig_status dig_gla_outgate_bwd(const void *o, const void *r, const float *ln_w, const float *ln_b, const void *dz,
                               void *d_o, void *d_r, float *dln_w, float *dln_b, long long rows, int d_v, float eps,
                               int dtype, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!o || !r || !dz || !d_o || !d_r) return DIG_ERR_INVALID_ARG;
    if (!aligned16(o) || !aligned16(r) || !aligned16(dz) || !aligned16(d_o) || !aligned16(d_r)) return DIG_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || !outgate_sizes_ok(rows, d_v, eps)) return DIG_ERR_INVALID_ARG;
    if (dln_w || dln_b) {
        const size_t need = outgate_bwd_workspace_bytes(rows, d_v);
        if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    }
    return launch_outgate_bwd(o, r, dz, ln_w, ln_b, d_o, d_r, dln_w, dln_b, rows, d_v, eps, dtype,
                              reinterpret_cast<float *>(workspace), (cudaStream_t)cuda_stream);
}

dig_status dig_gla_fwd_outgate(const void *q, const void *k, const void *v, const float *gate, const void *r,
                               const float *ln_w, const float *ln_b, float eps, void *out, void *z, int B, int H,
                               int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                               void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !r || !z) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(r) || !aligned16(z) ||
        (out && !aligned16(out)) || (ln_w && !aligned16(ln_w)) || (ln_b && !aligned16(ln_b)) || !(eps >= 0.f))
        return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype)) return DIG_ERR_INVALID_ARG;
    const size_t need = dig_gla_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 0);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    const int impl = choose_impl(d_k, d_v, chunk, dtype, false);
    if (impl < 0) return (dig_status)(-impl);
    GlaArgs a{};
    a.q = q; a.k = k; a.v = v; a.gate = gate;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, tile_chunk(impl, chunk), direction);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    // the plain forward pass (into z when the caller does not want `out`), then the gate kernel, which may
    // work in place
    a.out = out ? out : z;
    const dig_status st = impl == DIG_IMPL_TENSOR ? sweep_gla_fwd(a) : impl == DIG_IMPL_MMA ? mma_gla_fwd(a) : fma_gla_fwd(a);
    if (st != DIG_OK) return st;
    return launch_outgate_fwd_mixed(a.out, r, ln_w, ln_b, z, (long long)B * grid_h * grid_w * H, d_v, eps, dtype, a.stream);
}

size_t dig_gla_beta_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int dtype,
                                    int backward)
{
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, 0, dtype)) return 0;
    if (!mma_supports(d_k, d_v, chunk, dtype, backward != 0, true)) return 0;
    return mma_beta_workspace_bytes(make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, 0), backward != 0);
}

dig_status dig_gla_fwd_beta(const void *q, const void *k, const void *v, const float *gate, const float *bgate, void *out,
                            int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                            void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !bgate || !out) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(bgate) || !aligned16(out))
        return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype)) return DIG_ERR_INVALID_ARG;
    if (!mma_supports(d_k, d_v, chunk, dtype, false, true)) return DIG_ERR_UNSUPPORTED;
    const size_t need = dig_gla_beta_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 0);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    GlaArgs a{};
    a.bio.bgate = bgate;
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.out = out;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, direction);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return mma_gla_fwd(a);
}

dig_status dig_gla_bwd_beta(const void *q, const void *k, const void *v, const float *gate, const float *bgate,
                            const void *d_out, void *dq, void *dk, void *dv, float *dgate, float *dbgate,
                            int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int direction, int dtype,
                            void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !bgate || !d_out || !dq || !dk || !dv || !dgate || !dbgate) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(bgate) ||
        !aligned16(d_out) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(dgate) || !aligned16(dbgate))
        return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, direction, dtype)) return DIG_ERR_INVALID_ARG;
    if (!mma_supports(d_k, d_v, chunk, dtype, true, true)) return DIG_ERR_UNSUPPORTED;
    const size_t need = dig_gla_beta_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 1);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    GlaArgs a{};
    a.bio.bgate = bgate; a.bio.dbgate = dbgate;
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.d_out = d_out;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dgate = dgate;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, direction);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return mma_gla_bwd(a);
}

size_t dig_gla_multi_workspace_bytes(int B, int H, int grid_h, int grid_w, int d_k, int d_v, int chunk, int dtype,
                                     int backward)
{
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, 0, dtype)) return 0;
    if (!sweep_supports(d_k, d_v, chunk, dtype)) return 0;
    return sweep_multi_workspace_bytes(make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, 0), backward != 0, dtype);
}

dig_status dig_gla_fwd_multi(const void *q, const void *k, const void *v, const float *gate, void *out, int B, int H,
                             int grid_h, int grid_w, int d_k, int d_v, int chunk, unsigned direction_mask, int dtype,
                             void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !out) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(out)) return DIG_ERR_INVALID_ARG;
    if (direction_mask == 0 || direction_mask > 15u) return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, 0, dtype)) return DIG_ERR_INVALID_ARG;
    if (!sweep_supports(d_k, d_v, chunk, dtype)) return DIG_ERR_UNSUPPORTED;
    const size_t need = dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 0);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    GlaArgs a{};
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.out = out;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, 0);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return sweep_gla_fwd_multi(a, direction_mask);
}

dig_status dig_gla_bwd_multi(const void *q, const void *k, const void *v, const float *gate, const void *d_out,
                             void *dq, void *dk, void *dv, float *dgate, int B, int H, int grid_h, int grid_w, int d_k,
                             int d_v, int chunk, unsigned direction_mask, int dtype, void *workspace,
                             size_t workspace_bytes, void *cuda_stream)
{
    if (!q || !k || !v || !gate || !d_out || !dq || !dk || !dv || !dgate) return DIG_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(gate) || !aligned16(d_out) ||
        !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(dgate))
        return DIG_ERR_INVALID_ARG;
    if (direction_mask == 0 || direction_mask > 15u) return DIG_ERR_INVALID_ARG;
    if (!valid_geometry(B, H, grid_h, grid_w, d_k, d_v, chunk, 0, dtype)) return DIG_ERR_INVALID_ARG;
    if (!sweep_supports(d_k, d_v, chunk, dtype)) return DIG_ERR_UNSUPPORTED;
    const size_t need = dig_gla_multi_workspace_bytes(B, H, grid_h, grid_w, d_k, d_v, chunk, dtype, 1);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return DIG_ERR_WORKSPACE;
    GlaArgs a{};
    a.q = q; a.k = k; a.v = v; a.gate = gate; a.d_out = d_out;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dgate = dgate;
    a.ws = reinterpret_cast<float *>(workspace);
    a.g = make_geom(B, H, grid_h, grid_w, d_k, d_v, chunk, 0);
    a.dtype = dtype;
    a.stream = (cudaStream_t)cuda_stream;
    return sweep_gla_bwd_multi(a, direction_mask);
}

dig_status dig_last_device_status(void *cuda_stream)
{
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return DIG_ERR_CUDA;
    int host = 0;
    if (cudaMemcpyFromSymbol(&host, g_device_status, sizeof(int)) != cudaSuccess) return DIG_ERR_CUDA;
    if (host != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return DIG_ERR_CUDA;
        return (host & 1) ? DIG_ERR_TIMEOUT : DIG_ERR_RANGE;          // bit 0: a wait expired; bit 1: gates out of range
    }
    return DIG_OK;
}

dig_status dig_selftest_wait_timeout(unsigned limit_us, void *cuda_stream)
{
    if (limit_us == 0 || limit_us > 100000u) return DIG_ERR_INVALID_ARG;
    int *status = device_status_ptr();
    if (!status) return DIG_ERR_CUDA;
    wait_that_expires<<<1, 32, 0, (cudaStream_t)cuda_stream>>>(status, (unsigned long long)limit_us * 1000ull);
    return cuda_ok(cudaGetLastError());
}

dig_status dig_profile_enable(int on)
{
    if (on) {
        g_prof.kernel_of.clear();
        for (int i = 0; i < KID_COUNT; ++i) g_prof.launches[i] = 0;
    }
    g_prof.on = on != 0;
    return DIG_OK;
}

int dig_profile_kernels(void) { return KID_COUNT; }

dig_status dig_profile_read(int index, char *name, int name_bytes, int *launches, float *total_ms)
{
    if (index < 0 || index >= KID_COUNT || !name || name_bytes <= 0 || !launches || !total_ms)
        return DIG_ERR_INVALID_ARG;
    std::strncpy(name, kKernelNames[index], (size_t)name_bytes - 1);
    name[name_bytes - 1] = 0;
    *launches = g_prof.launches[index];
    float sum = 0.f;
    for (size_t i = 0; i < g_prof.kernel_of.size(); ++i) {
        if (g_prof.kernel_of[i] != index) continue;
        if (cudaEventSynchronize(g_prof.ev[2 * i + 1]) != cudaSuccess) return DIG_ERR_CUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_prof.ev[2 * i], g_prof.ev[2 * i + 1]) != cudaSuccess) return DIG_ERR_CUDA;
        sum += ms;
    }
    *total_ms = sum;
    return DIG_OK;
}

const char *dig_status_string(int status)
{
    switch (status) {
        case DIG_OK: return "ok";
        case DIG_ERR_INVALID_ARG: return "invalid argument";
        case DIG_ERR_UNSUPPORTED: return "unsupported configuration";
        case DIG_ERR_WORKSPACE: return "workspace missing or too small";
        case DIG_ERR_CUDA: return "CUDA runtime error";
        case DIG_ERR_TIMEOUT: return "device-side wait timed out";
        case DIG_ERR_SCRATCH_LIMIT: return "problem exceeds the built-in scratch of dig_gla_fwd_static";
        case DIG_ERR_RANGE: return "gate decay inside a chunk exceeds the documented range";
    }
    return "unknown status";
}

}  // extern "C"
