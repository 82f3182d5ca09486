// Tensor-core kernel family for chunkwise gated linear attention on sm_100a (Eq. attn_gla
// evaluated chunk by chunk, Section 3.5): dispatch of the forward and backward pipelines.
// bf16 storage, d_k = d_v = 64, 64-token tiles (chunk = 64; chunk = 128 requests are evaluated with
// the same tiles).
//
// Why tf32 operands: the decayed operands q*exp(Lam), k*exp(-Lam), the masked scores and the
// chunk states are not bf16 numbers; rounding them to bf16 (8 significant bits) puts the maximum
// error at 2e-2 of the output RMS, at the parity bound, while tf32 (11 bits) stays near 3e-3 with
// the same fp32 accumulation.
//
//   forward : gla_tc_state.cu (U^T per chunk, gamma)  ->  state_scan_fwd  ->  gla_tc_out.cu
//   backward: gla_tc_state.cu (U, W per chunk, gamma) ->  state_scan_bwd_tiles (both scans, carry)
//             ->  gla_tc_bwd.cu
// Per-chunk states live in the caller's workspace in the swizzled tile order of their consumers.
#include "dig_common.cuh"

namespace dig {

bool tensor_supports(int dk, int dv, int chunk, int dtype, bool backward)
{
    (void)backward;
    if (dtype != DIG_BF16 && dtype != DIG_BF16_F32OUT) return false;
    return dk == 64 && dv == 64 && (chunk == 64 || chunk == 128);      // 128: served with 64-token tiles
}

dig_status tensor_gla_fwd(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, false);
    int *status = device_status_ptr();
    const int sms = device_sm_count();
    if (!status || sms <= 0) return DIG_ERR_CUDA;
    if ((long long)g.B * g.H * g.N > (1ll << 30)) return DIG_ERR_UNSUPPORTED;      // chunk ids are 32-bit
    dig_status st;
    if ((st = launch_tc_state(a, w, false, sms, status)) != DIG_OK) return st;
    if ((st = launch_state_scan_fwd(w, g, a.stream, a.sio, true)) != DIG_OK) return st;
    return launch_tc_out(a, w, sms, status);
}

dig_status tensor_gla_bwd(const GlaArgs &a)
{
    const Geom &g = a.g;
    const Workspace w = carve_workspace(a.ws, g, true);
    int *status = device_status_ptr();
    const int sms = device_sm_count();
    if (!status || sms <= 0) return DIG_ERR_CUDA;
    if ((long long)g.B * g.H * g.N > (1ll << 30)) return DIG_ERR_UNSUPPORTED;
    dig_status st;
    if ((st = launch_tc_state(a, w, true, sms, status)) != DIG_OK) return st;
    if ((st = launch_state_scan_bwd_tiles(w, g, a.stream, a.sio)) != DIG_OK) return st;
    return launch_tc_bwd(a, w, sms, status);
}

}  // namespace dig
