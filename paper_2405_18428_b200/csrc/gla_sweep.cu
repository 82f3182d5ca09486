// tcgen05 "sweep" kernels of chunkwise gated linear attention (Eq. attn_gla, Section 3.5): the
// recurrence S_t = diag(exp(a_t)) S_{t-1} + k_t^T v_t, o_t = q_t S_t worked in 64-token tiles, with
// the d_k x d_v state held on chip while a CTA walks over a segment of consecutive tiles.
//
// A sequence of N tiles is cut into segments of G tiles; one CTA sweeps one segment.
//   forward : sweep_local  per segment, from a zero state: the state it leaves and its total decay
//             seg_scan     per sequence, over the few segment ends: the state entering each segment
//             sweep_fwd    per segment, from its true entry state: out = tril(Qc Kc^T) V + Qc Sc per tile
//   backward: sweep_local  (backward flavour) also stores, per (sub-)chunk, the zero-start state in
//                          fp16 and the decay since the segment start, and accumulates the segment's
//                          contribution to the state gradient
//             seg_scan     forward over the states, backward over the state gradients, gate-gradient carry
//             sweep_bwd    per segment in reverse: dq, dk, dv, dgate with the state gradient on chip
// With at least as many sequences as CTAs stay resident the sequences are not cut (one segment each):
// the forward pass is then sweep_fwd alone, started from the start state, and the backward pass runs a
// local sweep that only stores the per-chunk states.
// Per (sub-)chunk, with Lam the cumulative gate inside it, c = Lam_end / 2 per channel,
//   Qc = q exp(Lam - c), Kc = k exp(c - Lam), Sc = diag(exp(c)) S_in, Dc = diag(exp(c)) D_out:
//   P   = tril(Qc Kc^T)                         dP = tril(dO V^T)
//   out = P V + Qc Sc                           S_out = exp(2c) S_in + exp(c) (Kc^T V)
//   dq  = (dP Kc + dO Sc^T) exp(Lam - c)        dk = (dP^T Qc + V Dc^T) exp(c - Lam)
//   dv  = P^T dO + Kc Dc                        D_in = exp(2c) D_out + exp(c) (Qc^T dO)
//   dgate_j = sum_{r >= j} (q dq - k dk)_r  (running over the whole sequence in reverse scan order)
// In the backward sweep S_in = S_local + diag(G) S_segment, G the decay since the segment start, so
// dO Sc^T = dO Sc_local^T + (dO S_segment^T) diag(exp(c) G): two products and one fused multiply-add.
//
// Every product is a tcgen05.mma (kind::f16, fp16 operands, fp32 accumulators in tensor memory)
// issued by lane 0 of the last warp, which otherwise works like the others: all threads build operand tiles, mask
// the scores and post-process accumulators, phase by phase.  Token rows of the next tile are
// prefetched into registers; at d = 64 two CTAs of 256 threads share an SM, so one builds while the
// other's products are in the tensor pipe.
#include "sweep.cuh"

namespace dig {
namespace {

using namespace sw;

struct SweepArgs {
    const bf16 *q, *k, *v, *d_out;
    const float *gate;
    void *out, *dq, *dk, *dv;
    float *dgate;
    float *seg_state, *seg_gamma, *seg_dstate, *seg_carry;
    __half *seg_state16, *slot_s;
    float *slot_g;
    const float *s_in;      // forward pass with uncut sequences: the start state ([B*H][d][d], may be null) ...
    float *s_out;           // ... and where the final state goes (may be null)
    int *status;
    int accumulate;
    Geom g;
    Plan plan;
};

// ---- shared phases ------------------------------------------------------------------------------
__device__ __forceinline__ void cta_setup(Ctl *ctl, int nbar, uint32_t tmem_cols, char *tiles, int tile_bytes)
{
    const int tid = threadIdx.x;
    if (tid < 32) tmem_alloc(&ctl->tmem_base, tmem_cols);
    if (tid == 32) {
        for (int i = 0; i < nbar; ++i) mbar_init(&ctl->bar[i], 1);
        fence_barrier_init();
    }
    zero_smem(tiles, tile_bytes);
    fence_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}
__device__ __forceinline__ void cta_teardown(Ctl *ctl, uint32_t tmem_cols)
{
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(ctl->tmem_base, tmem_cols);
}

// Operand tiles of rows [lo, hi) of the prefetched tile (the other rows are zero):
//   tK <- k 2^(off - Lam), tV <- v, and where present tQ <- q 2^(Lam - off), tG <- dO.
__device__ __forceinline__ uint4 keep4(const uint4 &u, uint32_t m) { return make_uint4(u.x & m, u.y & m, u.z & m, u.w & m); }
template <int D, int NT, bool HQ, bool HD>
__device__ __forceinline__ void build_tiles(const Raw<Lay<D, NT>::NIT, HQ, HD> &r, char *tQ, char *tK, char *tV, char *tG,
                                            const float *table, const float *off, const int *row_off, int lo, int hi)
{
    using C = Cfg<D>;
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NIT; ++i) {
        const int it = (int)threadIdx.x + NT * i;
        if (item_exists<D, NT>(it)) {
            const int row = it / C::NCH, j = it - row * C::NCH;
            const int o = j * C::CHT + row * 16;
            // rows outside the sub-chunk or past the end of the sequence become zeros: no branch, a mask on the
            // packed result (which also discards whatever an out-of-range exponent produced there)
            const uint32_t m = (row >= lo && row < hi && row_off[row] >= 0) ? 0xffffffffu : 0u;
            float lam[8], of[8], x[8], y[8];
            ld8(table + row * C::LAMP + 8 * j, lam);
            ld8(off + 8 * j, of);
#pragma unroll
            for (int e = 0; e < 8; ++e) lam[e] -= of[e];
            unpack_b8(r.k[i], x);
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = x[e] * ex2(-lam[e]);
            *reinterpret_cast<uint4 *>(tK + o) = keep4(pack_h8(y), m);
            unpack_b8(r.v[i], x);
            *reinterpret_cast<uint4 *>(tV + o) = keep4(pack_h8(x), m);
            if (HQ) {
                unpack_b8(r.q[i], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) y[e] = x[e] * ex2(lam[e]);
                *reinterpret_cast<uint4 *>(tQ + o) = keep4(pack_h8(y), m);
            }
            if (HD) {
                unpack_b8(r.d[i], x);
                *reinterpret_cast<uint4 *>(tG + o) = keep4(pack_h8(x), m);
            }
        }
    }
}

// State product with channels along M: acc <- A^T B, A and B token tiles read down their rows
// (contraction over the 64 tokens).  Small heads: two value-column halves into the two lane halves.
template <int D>
__device__ __forceinline__ void issue_state_product(uint32_t tmem_acc, const char *tA, const char *tB)
{
    using C = Cfg<D>;
    const uint32_t a = smem_u32(tA), b = smem_u32(tB);
    if constexpr (C::BIGM) {
        issue<128, C::NACC, true, true, T / 16, C::CHT, C::CHT>(tmem_acc, a, b, false);
    } else {
        constexpr int HCH = C::NCH / 2;
        issue<64, D / 2, true, true, T / 16, C::CHT, C::CHT>(tmem_acc, a, b, false);
        issue<64, D / 2, true, true, T / 16, C::CHT, C::CHT>(tmem_acc + (16u << 16), a, b + HCH * C::CHT, false);
    }
}

// Bounded wait whose verdict is uniform over the warp (tcgen05.ld must never run under a
// lane-divergent condition).
__device__ __forceinline__ bool wait_all(uint64_t *bar, uint32_t parity, int *status)
{
    return __all_sync(0xffffffffu, mbar_wait(bar, parity, status)) != 0;
}

#define SYNC_OR_DIE()                               \
    do {                                            \
        if (!__syncthreads_and(ok)) goto die;       \
    } while (0)

// =================================================================================================
// sweep_local: a segment from a zero state.
// =================================================================================================
template <int D, int NT, bool BWD>
struct LocalSmem {
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    static constexpr int kTiles = (BWD ? 4 : 2) * C::TILE_T;
    // an M = 128 operand read down the rows of tQ / tK covers 16 chunks (more than the tile has): the
    // bytes behind it belong to the next tile, which is mapped and holds finite fp16 values
    static constexpr int kTilesPad = kTiles;
    static_assert(!C::BIGM || 16 * C::CHT <= 2 * C::TILE_T, "an M = 128 operand must stay inside the tile area");
    static constexpr int kFloats = T * C::LAMP + L::NSEG * D + 8 * D;
    static constexpr size_t bytes = kTilesPad + kFloats * 4 + 4 * T * 4 + sizeof(Ctl);
    static constexpr uint32_t tmem_cols = C::BIGM ? (BWD ? 256 : 128) : (BWD ? 64 : 32);
};

// SLOTS: also store, per (sub-)chunk, the zero-start state and the decay since the segment start (what the
// backward sweep reads).  The backward flavour (BWD) always does and adds the segment's contribution to the
// state gradient; a backward pass over uncut sequences needs only the stored states (BWD = false, SLOTS = true).
template <int D, int NT, bool BWD, int OCC, bool SLOTS = BWD>
__global__ void __launch_bounds__(NT, OCC)
sweep_local(const SweepArgs a)
{
    static_assert(SLOTS || !BWD, "the backward flavour stores the per-chunk states");
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    using SM = LocalSmem<D, NT, BWD>;
    extern __shared__ __align__(128) char smem[];
    char *tQ = smem, *tK = BWD ? tQ + C::TILE_T : smem, *tV = tK + C::TILE_T, *tG = tV + C::TILE_T;
    float *table = reinterpret_cast<float *>(smem + SM::kTilesPad);
    float *sTot = table + T * C::LAMP, *vecb = sTot + L::NSEG * D;
    int *rowOff = reinterpret_cast<int *>(vecb + 8 * D);
    Ctl *ctl = reinterpret_cast<Ctl *>(rowOff + 4 * T);
    constexpr uint32_t aU = 0, aW = C::BIGM ? C::NACC : D / 2;

    const int tid = threadIdx.x;
    constexpr int kIssuer = NT - 32;        // lane 0 of the last warp issues the MMAs (warps 0 and 1 carry the per-channel work)
    cta_setup(ctl, 1, SM::tmem_cols, smem, SM::kTilesPad);
    const uint32_t tmem = ctl->tmem_base, lane_base = (uint32_t)(32 * ((tid >> 5) & 3)) << 16;
    const Geom &g = a.g;
    const Plan &pl = a.plan;
    const StateMap<D, NT> sm;
    float S[L::NPS][8], Wl[L::NPS][8];
    Raw<L::NIT, BWD, BWD> raw;
    float gcum = 0.f;
    uint32_t par = 0;
    bool ok = true;
    int cur = 0, iter = 0;
    const int total = g.B * g.H * pl.nseg;

    pdl_wait();
    pdl_launch_dependents();
    for (int sid = blockIdx.x; sid < total; sid += gridDim.x) {
        const int bh = sid / pl.nseg, sg = sid - bh * pl.nseg, b = bh / g.H, h = bh - b * g.H;
        const int t0 = sg * pl.G, t1 = min(t0 + pl.G, pl.ntile);
        load_state<D, NT>(nullptr, sm, S);
        if (BWD) load_state<D, NT>(nullptr, sm, Wl);
        gcum = 0.f;
        if (tid < T) rowOff[cur * T + tid] = tile_row_offset(g, b, h, D, t0, tid);
        __syncthreads();
        load_raw<D, NT, BWD, BWD>(raw, a.q, a.k, a.v, a.d_out, a.gate, rowOff + cur * T);
        for (int tile = t0; tile < t1; ++tile) {
            const int nrow = min(T, g.L - tile * T), nxt = (cur + 1) & 3;
            if (tid < T) {
                rowOff[nxt * T + tid] = tile + 1 < t1 ? tile_row_offset(g, b, h, D, tile + 1, tid) : -1;
                // this kernel's tiles are short: the register prefetch alone does not cover the memory latency
                if (tile + 2 < t1) prefetch_row<D, BWD, BWD>(a.q, a.k, a.v, a.d_out, a.gate, tile_row_offset(g, b, h, D, tile + 2, tid));
            }
            write_gates<D, NT, BWD, BWD>(raw, table, rowOff + cur * T);
            __syncthreads();
            // the vectors of an undivided tile are written inside the prefix pass (no barrier of their own)
            const bool whole_ok = pl.sub_max == T;
            const Vec v0 = vec_of<D>(vecb, iter & 1);
            float tot_c = 0.f;
            const bool need = gate_prefix<D, NT>(table, sTot, tot_c, [&](int c, float t) {
                if (whole_ok) {
                    const float cv = 0.5f * t;
                    v0.off[c] = cv;
                    v0.ec[c] = ex2(cv);
                    v0.e2c[c] = ex2(t);
                    if (BWD) v0.aux[c] = ex2(gcum + cv);
                }
            });
            const bool whole = whole_ok && !need;
            int s = pl.sub_max;
            if (need || s < T) {
                bool bad;
                s = choose_sub<D>(table, need ? min(s, T / 2) : s, &bad);
                if (bad && tid == 0) atomicOr(a.status, kStatusRange);
            }
            const int nsub = (nrow + s - 1) / s;
            for (int u = 0; u < nsub; ++u, ++iter) {
                const int lo = u * s, hi = min(lo + s, T);
                const Vec vc = vec_of<D>(vecb, iter & 1);
                if (tid < D) {
                    float t = tot_c;
                    if (!whole) {
                        const float base = lo ? table[(lo - 1) * C::LAMP + tid] : 0.f;
                        t = table[(hi - 1) * C::LAMP + tid] - base;
                        const float cv = 0.5f * t;
                        vc.off[tid] = base + cv;
                        vc.ec[tid] = ex2(cv);
                        vc.e2c[tid] = ex2(t);
                        if (BWD) vc.aux[tid] = ex2(gcum + cv);  // decay from the segment start to the sub-chunk's centre
                    }
                    if (SLOTS) {
                        const size_t slot = ((size_t)(nsub - 1 - u) * g.B * g.H + bh) * pl.ntile + tile;
                        a.slot_g[slot * D + tid] = gcum;
                    }
                    gcum += t;
                }
                if (!whole) __syncthreads();
                {
                    build_tiles<D, NT, BWD, BWD>(raw, tQ, tK, tV, tG, table, vc.off, rowOff + cur * T, lo, min(hi, nrow));
                    if (SLOTS) {
                        const size_t slot = ((size_t)(nsub - 1 - u) * g.B * g.H + bh) * pl.ntile + tile;
                        write_state_slot<D, NT>(a.slot_s + slot * (D * D), sm, S, vc.ec);
                    }
                    fence_async_smem();
                }
                tc_fence_before_sync();
                SYNC_OR_DIE();
                if (tid == kIssuer) {
                    tc_fence_after_sync();
                    issue_state_product<D>(tmem + aU, tK, tV);                   // Kc^T V
                    if (BWD) issue_state_product<D>(tmem + aW, tQ, tG);         // Qc^T dO
                    mma_commit(&ctl->bar[0]);
                }
                {
                    if (u == nsub - 1 && tile + 1 < t1)
                        load_raw<D, NT, BWD, BWD>(raw, a.q, a.k, a.v, a.d_out, a.gate, rowOff + nxt * T);
                    ok = wait_all(&ctl->bar[0], par, a.status);
                    if (ok) {
                        tc_fence_after_sync();
                        update_state<D, NT>(lane_base, tmem + aU, sm, S, vc.e2c, vc.ec);
                        if (BWD) {
                            // W_segment += (decay since the segment start) * exp(c) * (Qc^T dO)
                            const float fs = sm.valid ? vc.aux[sm.c] : 0.f;
#pragma unroll
                            for (int i = 0; i < L::NPS; ++i)
                                if (sm.has(i)) {
                                    float w[8];
                                    tmem_ld8(lane_base + tmem + aW + sm.tcol(i), w);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) Wl[i][e] += fs * w[e];
                                }
                        }
                    }
                    tc_fence_before_sync();
                }
                par ^= 1;
            }
            cur = nxt;
        }
        {
            store_state<D, NT>(a.seg_state + (size_t)sid * D * D, sm, S);
            if (BWD) store_state<D, NT>(a.seg_dstate + (size_t)sid * D * D, sm, Wl);
            if (tid < D) a.seg_gamma[(size_t)sid * D + tid] = gcum;
        }
    }
die:
    cta_teardown(ctl, SM::tmem_cols);
}

// =================================================================================================
// seg_scan: the recurrence over segment ends, one sequence per blockIdx.x, 8 state rows per block,
// 8 lanes per row.  Forward: seg_state[s] (state a segment leaves from a zero start) becomes the
// state entering segment s.  Backward flavour: seg_dstate[s] (the segment's own contribution)
// becomes the gradient with respect to the state leaving segment s, seg_carry the gate-gradient
// carried into the segment from later ones, seg_state16 an fp16 copy of the entry states in the
// dense chunk-major order the backward sweep bulk-copies.
// =================================================================================================
template <int D, bool BWD>
__global__ void __launch_bounds__(64)
seg_scan(float *seg_state, const float *seg_gamma, float *seg_dstate, float *seg_carry, __half *seg_state16,
         const float *s_in, float *s_out, const float *ds_out, float *ds_in, int nseg)
{
    constexpr int NV = (D / 4 + 7) / 8;               // float4 pieces per lane
    constexpr int NB = NV <= 2 ? 8 : 4;               // segments whose loads are in flight together
    const int bh = blockIdx.x, c = blockIdx.y * 8 + (threadIdx.x >> 3), l8 = threadIdx.x & 7;
    pdl_wait();
    pdl_launch_dependents();
    float4 s[NV];
    const size_t row = (size_t)c * D;
    const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int e = 4 * (l8 + 8 * i);
        s[i] = (s_in && e < D) ? *reinterpret_cast<const float4 *>(s_in + (size_t)bh * D * D + row + e) : zero4;
    }
    for (int sg0 = 0; sg0 < nseg; sg0 += NB) {
        float4 t[NB][NV];
        float gam[NB];
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            const int sg = min(sg0 + j, nseg - 1);
            gam[j] = seg_gamma[((size_t)bh * nseg + sg) * D + c];
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int e = 4 * (l8 + 8 * i);
                t[j][i] = e < D ? *reinterpret_cast<const float4 *>(seg_state + ((size_t)bh * nseg + sg) * D * D + row + e) : zero4;
            }
        }
#pragma unroll
        for (int j = 0; j < NB; ++j) {
            const int sg = sg0 + j;
            if (sg < nseg) {
                const float gm = exp2f(gam[j]);
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int e = 4 * (l8 + 8 * i);
                    if (e < D) {
                        *reinterpret_cast<float4 *>(seg_state + ((size_t)bh * nseg + sg) * D * D + row + e) = s[i];
                        if (BWD) {
                            __half2 lo = __floats2half2_rn(s[i].x, s[i].y), hi = __floats2half2_rn(s[i].z, s[i].w);
                            uint2 pk;
                            pk.x = *reinterpret_cast<uint32_t *>(&lo);
                            pk.y = *reinterpret_cast<uint32_t *>(&hi);
                            char *dst = reinterpret_cast<char *>(seg_state16 + ((size_t)bh * nseg + sg) * D * D);
                            *reinterpret_cast<uint2 *>(dst + ((e >> 3) * D + c) * 16 + (e & 7) * 2) = pk;
                        }
                        s[i] = make_float4(gm * s[i].x + t[j][i].x, gm * s[i].y + t[j][i].y, gm * s[i].z + t[j][i].z,
                                           gm * s[i].w + t[j][i].w);
                    }
                }
            }
        }
    }
    if (s_out) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int e = 4 * (l8 + 8 * i);
            if (e < D) *reinterpret_cast<float4 *>(s_out + (size_t)bh * D * D + row + e) = s[i];
        }
    }
    if (BWD) {
        float4 d[NV];
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int e = 4 * (l8 + 8 * i);
            d[i] = (ds_out && e < D) ? *reinterpret_cast<const float4 *>(ds_out + (size_t)bh * D * D + row + e) : zero4;
        }
        // s holds the state leaving the last segment; walking back, it is replaced by the entry state of
        // the segment just handled, which is the state leaving the one before it
        for (int sg0 = nseg - 1; sg0 >= 0; sg0 -= NB) {
            float4 t[NB][NV], sp[NB][NV];
            float gam[NB];
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const int sg = max(sg0 - j, 0);
                gam[j] = seg_gamma[((size_t)bh * nseg + sg) * D + c];
#pragma unroll
                for (int i = 0; i < NV; ++i) {
                    const int e = 4 * (l8 + 8 * i);
                    t[j][i] = e < D ? *reinterpret_cast<const float4 *>(seg_dstate + ((size_t)bh * nseg + sg) * D * D + row + e) : zero4;
                    sp[j][i] = e < D ? *reinterpret_cast<const float4 *>(seg_state + ((size_t)bh * nseg + sg) * D * D + row + e) : zero4;
                }
            }
#pragma unroll
            for (int j = 0; j < NB; ++j) {
                const int sg = sg0 - j;
                if (sg >= 0) {
                    const float gm = exp2f(gam[j]);
                    float dot = 0.f;
#pragma unroll
                    for (int i = 0; i < NV; ++i) {
                        const int e = 4 * (l8 + 8 * i);
                        if (e < D) {
                            *reinterpret_cast<float4 *>(seg_dstate + ((size_t)bh * nseg + sg) * D * D + row + e) = d[i];
                            dot += s[i].x * d[i].x + s[i].y * d[i].y + s[i].z * d[i].z + s[i].w * d[i].w;
                            d[i] = make_float4(gm * d[i].x + t[j][i].x, gm * d[i].y + t[j][i].y, gm * d[i].z + t[j][i].z,
                                               gm * d[i].w + t[j][i].w);
                            s[i] = sp[j][i];
                        }
                    }
                    dot += __shfl_xor_sync(0xffffffffu, dot, 4);
                    dot += __shfl_xor_sync(0xffffffffu, dot, 2);
                    dot += __shfl_xor_sync(0xffffffffu, dot, 1);
                    if (l8 == 0) seg_carry[((size_t)bh * nseg + sg) * D + c] = dot;
                }
            }
        }
        if (ds_in) {
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const int e = 4 * (l8 + 8 * i);
                if (e < D) *reinterpret_cast<float4 *>(ds_in + (size_t)bh * D * D + row + e) = d[i];
            }
        }
    }
}

// =================================================================================================
// sweep_fwd: a segment from its entry state; writes out.
// =================================================================================================
template <int D, int NT>
struct FwdSmem {
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    static constexpr int kTiles = 3 * C::TILE_T + C::TILE_S + C::TILE_P;      // tQ tK tV tS tP
    static constexpr int kFloats = T * C::LAMP + L::NSEG * D + 8 * D;
    static constexpr size_t bytes = kTiles + kFloats * 4 + 4 * T * 4 + sizeof(Ctl);
    static constexpr uint32_t tmem_cols = C::BIGM ? 256 : 128;
};

template <int D, int NT, typename TO, int OCC>
__global__ void __launch_bounds__(NT, OCC)
sweep_fwd(const SweepArgs a)
{
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    using SM = FwdSmem<D, NT>;
    extern __shared__ __align__(128) char smem[];
    char *tQ = smem, *tK = tQ + C::TILE_T, *tV = tK + C::TILE_T, *tS = tV + C::TILE_T, *tP = tS + C::TILE_S;
    float *table = reinterpret_cast<float *>(smem + SM::kTiles);
    float *sTot = table + T * C::LAMP, *vecb = sTot + L::NSEG * D;
    int *rowOff = reinterpret_cast<int *>(vecb + 8 * D);
    Ctl *ctl = reinterpret_cast<Ctl *>(rowOff + 4 * T);
    // the state product is issued after the scores have been read and reuses their columns
    constexpr uint32_t aP = 0, aO = C::BIGM ? C::NACC : 64, aU = aP;
    static_assert(aO + C::NACC <= SM::tmem_cols, "tensor memory");

    const int tid = threadIdx.x, lane = tid & 31, q4 = (tid >> 5) & 3, cg = tid >> 7, hf = lane >> 4;
    constexpr int kIssuer = NT - 32;        // lane 0 of the last warp issues the MMAs (warps 0 and 1 carry the per-channel work)
    const int r16 = 16 * q4 + (lane & 15);
    cta_setup(ctl, 1, SM::tmem_cols, smem, SM::kTiles);
    const uint32_t tmem = ctl->tmem_base, lane_base = (uint32_t)(32 * q4) << 16;
    const Geom &g = a.g;
    const Plan &pl = a.plan;
    const StateMap<D, NT> sm;
    float S[L::NPS][8];
    Raw<L::NIT, true, false> raw;
    uint32_t par = 0;
    bool ok = true;
    int cur = 0, iter = 0;
    const int total = g.B * g.H * pl.nseg;
    TO *out = reinterpret_cast<TO *>(a.out);

    // The first tile's rows are inputs of the call: their loads need not wait for the scan kernel (whose own
    // wait covered whatever produced them).  Uncut sequences have no kernel in front that has waited: wait first.
    if (pl.nseg == 1) pdl_wait();
    {
        const int sid = blockIdx.x;
        if (sid < total) {
            const int bh = sid / pl.nseg, sg = sid - bh * pl.nseg, b = bh / g.H, h = bh - b * g.H;
            if (tid < T) rowOff[cur * T + tid] = tile_row_offset(g, b, h, D, sg * pl.G, tid);
            __syncthreads();
            load_raw<D, NT, true, false>(raw, a.q, a.k, a.v, nullptr, a.gate, rowOff + cur * T);
        }
    }
    pdl_wait();
    pdl_launch_dependents();
    for (int sid = blockIdx.x; sid < total; sid += gridDim.x) {
        const int bh = sid / pl.nseg, sg = sid - bh * pl.nseg, b = bh / g.H, h = bh - b * g.H;
        const int t0 = sg * pl.G, t1 = min(t0 + pl.G, pl.ntile);
        if (pl.nseg == 1) load_state<D, NT>(a.s_in ? a.s_in + (size_t)sid * D * D : nullptr, sm, S);      // uncut: no scan ran
        else load_state<D, NT>(a.seg_state + (size_t)sid * D * D, sm, S);
        if (sid != (int)blockIdx.x) {
            if (tid < T) rowOff[cur * T + tid] = tile_row_offset(g, b, h, D, t0, tid);
            __syncthreads();
            load_raw<D, NT, true, false>(raw, a.q, a.k, a.v, nullptr, a.gate, rowOff + cur * T);
        }
        for (int tile = t0; tile < t1; ++tile) {
            const int nrow = min(T, g.L - tile * T), nxt = (cur + 1) & 3;
            if (tid < T) rowOff[nxt * T + tid] = tile + 1 < t1 ? tile_row_offset(g, b, h, D, tile + 1, tid) : -1;
            write_gates<D, NT, true, false>(raw, table, rowOff + cur * T);
            __syncthreads();
            const int my_off = rowOff[cur * T + r16];
            // the vectors of an undivided tile are written inside the prefix pass (no barrier of their own)
            const bool whole_ok = pl.sub_max == T;
            const Vec v0 = vec_of<D>(vecb, iter & 1);
            float tot_c = 0.f;
            const bool need = gate_prefix<D, NT>(table, sTot, tot_c, [&](int c, float t) {
                if (whole_ok) {
                    const float cv = 0.5f * t;
                    v0.off[c] = cv;
                    v0.ec[c] = ex2(cv);
                    v0.e2c[c] = ex2(t);
                }
            });
            const bool whole = whole_ok && !need;
            int s = pl.sub_max;
            if (need || s < T) {
                bool bad;
                s = choose_sub<D>(table, need ? min(s, T / 2) : s, &bad);
                if (bad && tid == 0) atomicOr(a.status, kStatusRange);
            }
            const int nsub = (nrow + s - 1) / s;
            for (int u = 0; u < nsub; ++u, ++iter) {
                const int lo = u * s, hi = min(lo + s, T);
                const Vec vc = vec_of<D>(vecb, iter & 1);
                if (!whole) {
                    if (tid < D) {
                        const float base = lo ? table[(lo - 1) * C::LAMP + tid] : 0.f;
                        const float t = table[(hi - 1) * C::LAMP + tid] - base, cv = 0.5f * t;
                        vc.off[tid] = base + cv;
                        vc.ec[tid] = ex2(cv);
                        vc.e2c[tid] = ex2(t);
                    }
                    __syncthreads();
                }
                {
                    build_tiles<D, NT, true, false>(raw, tQ, tK, tV, nullptr, table, vc.off, rowOff + cur * T, lo, min(hi, nrow));
                    write_state_tile<D, NT>(tS, sm, S, vc.ec);                       // Sc = diag(2^c) S
                    fence_async_smem();
                }
                tc_fence_before_sync();
                SYNC_OR_DIE();
                if (tid == kIssuer) {
                    tc_fence_after_sync();
                    issue<64, 64, false, false, C::KS, C::CHT, C::CHT>(tmem + aP, smem_u32(tQ), smem_u32(tK), false);   // Qc Kc^T
                    mma_commit(&ctl->bar[0]);
                    issue<64, D, false, true, C::KS, C::CHT, C::CHS>(tmem + aO, smem_u32(tQ), smem_u32(tS), false);     // Qc Sc
                }
                {
                    if (u == nsub - 1 && tile + 1 < t1)
                        load_raw<D, NT, true, false>(raw, a.q, a.k, a.v, nullptr, a.gate, rowOff + nxt * T);
                    ok = wait_all(&ctl->bar[0], 0, a.status);          // completes twice per iteration: parities 0, 1
                    if (ok) {
                        tc_fence_after_sync();
                        // scores of row r16 (lanes 0-15 hold accumulator rows): keep s <= t, the diagonal has weight 1.
                        // Column chunks entirely above the diagonal for all 16 rows of the warp are never written (the
                        // tile starts out zero), chunks entirely below it need no selects.
#pragma unroll
                        for (int i = 0; i < L::NPT; ++i) {
                            const int sc = cg + L::NCG * i;
                            if (sc < T / 8 && 8 * sc <= 16 * q4 + 15) {           // uniform over the warp
                                float p[8];
                                tmem_ld8(lane_base + tmem + aP + 8 * sc, p);
                                if (8 * sc + 7 > 16 * q4) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) p[e] = (8 * sc + e <= r16) ? p[e] : 0.f;
                                }
                                if (hf == 0) *reinterpret_cast<uint4 *>(tP + sc * C::CHT + r16 * 16) = pack_h8(p);
                            }
                        }
                    }
                    fence_async_smem();
                }
                tc_fence_before_sync();
                SYNC_OR_DIE();
                if (tid == kIssuer) {
                    tc_fence_after_sync();
                    issue<64, D, false, true, T / 16, C::CHT, C::CHT>(tmem + aO, smem_u32(tP), smem_u32(tV), true);     // + P V
                    issue_state_product<D>(tmem + aU, tK, tV);                                                         // Kc^T V
                    mma_commit(&ctl->bar[0]);
                }
                {
                    ok = wait_all(&ctl->bar[0], 1, a.status);
                    if (ok) {
                        tc_fence_after_sync();
                        update_state<D, NT>(lane_base, tmem + aU, sm, S, vc.e2c, vc.ec);
                        const bool inrow = hf == 0 && r16 >= lo && r16 < hi && my_off >= 0;
                        const size_t ro = (size_t)(my_off < 0 ? 0 : my_off);
#pragma unroll
                        for (int i = 0; i < L::NPC; ++i) {
                            const int jc = cg + L::NCG * i;
                            if (jc < C::NCH) {
                                float o[8];
                                tmem_ld8(lane_base + tmem + aO + 8 * jc, o);
                                if (inrow) store_out8(out + ro + 8 * jc, o, a.accumulate != 0);
                            }
                        }
                    }
                    tc_fence_before_sync();
                }
                par ^= 1;
            }
            cur = nxt;
        }
        if (pl.nseg == 1 && a.s_out) store_state<D, NT>(a.s_out + (size_t)sid * D * D, sm, S);
    }
die:
    cta_teardown(ctl, SM::tmem_cols);
}

// =================================================================================================
// sweep_bwd: a segment in reverse scan order with the state gradient on chip.
// =================================================================================================
template <int D, int NT>
struct BwdSmem {
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    static constexpr int kTiles = 4 * C::TILE_T + 3 * C::TILE_S + 2 * C::TILE_P;      // tQ tK tV tG | tS tI tD | tP tdP
    static constexpr int kFloats = T * C::LAMP + L::NSEG * D + 8 * D + 2 * D;
    static constexpr size_t bytes = kTiles + kFloats * 4 + 4 * T * 4 + sizeof(Ctl);
    static constexpr uint32_t tmem_cols = 256;
};

template <int D, int NT, typename TO, int OCC>
__global__ void __launch_bounds__(NT, OCC)
sweep_bwd(const SweepArgs a)
{
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    using SM = BwdSmem<D, NT>;
    extern __shared__ __align__(128) char smem[];
    char *tQ = smem, *tK = tQ + C::TILE_T, *tV = tK + C::TILE_T, *tG = tV + C::TILE_T;
    char *tS = tG + C::TILE_T, *tI = tS + C::TILE_S, *tD = tI + C::TILE_S;
    char *tP = tD + C::TILE_S, *tdP = tP + C::TILE_P;
    float *table = reinterpret_cast<float *>(smem + SM::kTiles);
    float *sTot = table + T * C::LAMP, *vecb = sTot + L::NSEG * D, *sCarry = vecb + 8 * D;
    int *rowOff = reinterpret_cast<int *>(sCarry + 2 * D);
    Ctl *ctl = reinterpret_cast<Ctl *>(rowOff + 4 * T);
    constexpr uint32_t W0 = C::BIGM ? C::NACC : 64;
    constexpr uint32_t aP = 0, aQK = W0, aV = W0 + C::NACC, kHi = 16u << 16;
    static_assert(aV + C::NACC <= SM::tmem_cols, "tensor memory");

    const int tid = threadIdx.x, lane = tid & 31, q4 = (tid >> 5) & 3, cg = tid >> 7, hf = lane >> 4;
    constexpr int kIssuer = NT - 32;        // lane 0 of the last warp issues the MMAs (warps 0 and 1 carry the per-channel work)
    const int r16 = 16 * q4 + (lane & 15);
    cta_setup(ctl, 2, SM::tmem_cols, smem, SM::kTiles);
    const uint32_t tmem = ctl->tmem_base, lane_base = (uint32_t)(32 * q4) << 16;
    uint64_t *barG1 = &ctl->bar[0], *barS = &ctl->bar[1];
    const Geom &g = a.g;
    const Plan &pl = a.plan;
    const StateMap<D, NT> sm;
    float Dst[L::NPS][8];
    Raw<L::NIT, true, true> raw;
    uint32_t par = 0;
    bool ok = true;
    int cur = 0, iter = 0, cpar = 0;
    const int total = g.B * g.H * pl.nseg;
    TO *dq = reinterpret_cast<TO *>(a.dq), *dk = reinterpret_cast<TO *>(a.dk), *dv = reinterpret_cast<TO *>(a.dv);

    // the first tile's rows are inputs of the call: their loads need not wait for the scan kernel
    auto prime = [&](int sid) {
        const int bh = sid / pl.nseg, sg = sid - bh * pl.nseg, b = bh / g.H, h = bh - b * g.H;
        const int t1 = min(sg * pl.G + pl.G, pl.ntile);
        if (tid < T) rowOff[cur * T + tid] = tile_row_offset(g, b, h, D, t1 - 1, tid);
        __syncthreads();
        load_raw<D, NT, true, true>(raw, a.q, a.k, a.v, a.d_out, a.gate, rowOff + cur * T);
    };
    if ((int)blockIdx.x < total) prime(blockIdx.x);
    pdl_wait();
    pdl_launch_dependents();
    for (int sid = blockIdx.x; sid < total; sid += gridDim.x) {
        const int bh = sid / pl.nseg, sg = sid - bh * pl.nseg, b = bh / g.H, h = bh - b * g.H;
        const int t0 = sg * pl.G, t1 = min(t0 + pl.G, pl.ntile);
        load_state<D, NT>(a.seg_dstate + (size_t)sid * D * D, sm, Dst);
        if (tid < D) sCarry[cpar * D + tid] = a.seg_carry[(size_t)sid * D + tid];
        if (sid != (int)blockIdx.x) prime(sid);
        if (tid == kIssuer) {
            // the zero-start state of the sub-chunk worked first (always slot 0 of its tile) and, once per
            // segment, the state entering the segment; later sub-chunks' states are fetched as soon as the
            // products of the one before are done
            const char *src = reinterpret_cast<const char *>(a.slot_s + ((size_t)bh * pl.ntile + (t1 - 1)) * (D * D));
            const char *seg16 = reinterpret_cast<const char *>(a.seg_state16 + (size_t)sid * D * D);
            mbar_arrive_expect_tx(barS, 2u * C::NCH * D * 16u);
            for (int j = 0; j < C::NCH; ++j) {
                bulk_g2s(tS + j * C::CHS, src + j * D * 16, D * 16, barS);
                bulk_g2s(tI + j * C::CHS, seg16 + j * D * 16, D * 16, barS);
            }
        }
        for (int tile = t1 - 1; tile >= t0; --tile) {
            const int nrow = min(T, g.L - tile * T), nxt = (cur + 1) & 3;
            if (tid < T) rowOff[nxt * T + tid] = tile > t0 ? tile_row_offset(g, b, h, D, tile - 1, tid) : -1;
            write_gates<D, NT, true, true>(raw, table, rowOff + cur * T);
            __syncthreads();
            const int my_off = rowOff[cur * T + r16];
            // decay since the segment start of the sub-chunk worked first (always slot 0): fetched ahead of its use
            const float g_first = tid < D ? a.slot_g[((size_t)bh * pl.ntile + tile) * D + tid] : 0.f;
            // the vectors of an undivided tile are written inside the prefix pass (no barrier of their own)
            const bool whole_ok = pl.sub_max == T;
            const Vec v0 = vec_of<D>(vecb, iter & 1);
            float tot_c = 0.f;
            const bool need = gate_prefix<D, NT>(table, sTot, tot_c, [&](int c, float t) {
                if (whole_ok) {
                    const float cv = 0.5f * t;
                    v0.off[c] = cv;
                    v0.ec[c] = ex2(cv);
                    v0.e2c[c] = ex2(t);
                    v0.aux[c] = ex2(cv + g_first);
                }
            });
            const bool whole = whole_ok && !need;
            int s = pl.sub_max;
            if (need || s < T) {
                bool bad;
                s = choose_sub<D>(table, need ? min(s, T / 2) : s, &bad);
                if (bad && tid == 0) atomicOr(a.status, kStatusRange);
            }
            const int nsub = (nrow + s - 1) / s;
            for (int u = nsub - 1; u >= 0; --u, ++iter) {
                const int lo = u * s, hi = min(lo + s, T), hiv = min(hi, nrow);
                const size_t slot = ((size_t)(nsub - 1 - u) * g.B * g.H + bh) * pl.ntile + tile;
                const Vec vc = vec_of<D>(vecb, iter & 1);
                if (!whole) {
                    if (tid < D) {
                        const float base = lo ? table[(lo - 1) * C::LAMP + tid] : 0.f;
                        const float t = table[(hi - 1) * C::LAMP + tid] - base, cv = 0.5f * t;
                        vc.off[tid] = base + cv;
                        vc.ec[tid] = ex2(cv);
                        vc.e2c[tid] = ex2(t);
                        vc.aux[tid] = ex2(cv + (u == nsub - 1 ? g_first : a.slot_g[slot * D + tid]));   // exp(c) * decay since the segment start
                    }
                    __syncthreads();
                }
                {
                    build_tiles<D, NT, true, true>(raw, tQ, tK, tV, tG, table, vc.off, rowOff + cur * T, lo, hiv);
                    write_state_tile<D, NT>(tD, sm, Dst, vc.ec);                    // Dc = diag(2^c) D
                    fence_async_smem();
                }
                tc_fence_before_sync();
                SYNC_OR_DIE();
                if (tid == kIssuer) {
                    ok = mbar_wait(barS, par, a.status);          // both state tiles have landed
                    tc_fence_after_sync();
                    const uint32_t sQ = smem_u32(tQ), sK = smem_u32(tK), sV = smem_u32(tV), sG = smem_u32(tG);
                    const uint32_t sS = smem_u32(tS), sI = smem_u32(tI), sD = smem_u32(tD);
                    issue<64, 64, false, false, C::KS, C::CHT, C::CHT>(tmem + aP, sQ, sK, false);             // Qc Kc^T
                    issue<64, 64, false, false, C::KS, C::CHT, C::CHT>(tmem + aP + kHi, sG, sV, false);       // dO V^T
                    mma_commit(barG1);
                    issue<64, D, false, false, C::KS, C::CHT, C::CHS>(tmem + aQK, sG, sS, false);             // dO Sc_local^T
                    issue<64, D, false, false, C::KS, C::CHT, C::CHS>(tmem + aV, sG, sI, false);              // dO S_segment^T
                    issue<64, D, false, false, C::KS, C::CHT, C::CHS>(tmem + aQK + kHi, sV, sD, false);       // V Dc^T
                    issue<64, D, false, true, C::KS, C::CHT, C::CHS>(tmem + aV + kHi, sK, sD, false);         // Kc Dc
                }
                {
                    // the raw rows are spent: the next tile's gates (needed first) start now, its q, k, v, dO rows
                    // after the epilogue, which needs the registers
                    if (u == 0 && tile > t0)
                        load_raw<D, NT, true, true, true, false>(raw, a.q, a.k, a.v, a.d_out, a.gate, rowOff + nxt * T);
                    ok = wait_all(barG1, 0, a.status);                 // completes twice per iteration: parities 0, 1
                    if (ok) {
                        tc_fence_after_sync();
                        // lanes 0-15: scores, lanes 16-31: dO V^T; keep s <= t, the diagonal has weight 1.  Column
                        // chunks entirely above the diagonal for all rows of the warp are never written (the tiles
                        // start out zero), chunks entirely below it need no selects.
#pragma unroll
                        for (int i = 0; i < L::NPT; ++i) {
                            const int sc = cg + L::NCG * i;
                            if (sc < T / 8 && 8 * sc <= 16 * q4 + 15) {           // uniform over the warp
                                float p[8];
                                tmem_ld8(lane_base + tmem + aP + 8 * sc, p);
                                if (8 * sc + 7 > 16 * q4) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) p[e] = (8 * sc + e <= r16) ? p[e] : 0.f;
                                }
                                *reinterpret_cast<uint4 *>((hf ? tdP : tP) + sc * C::CHT + r16 * 16) = pack_h8(p);
                            }
                        }
                    }
                    fence_async_smem();
                }
                tc_fence_before_sync();
                SYNC_OR_DIE();
                if (tid == kIssuer) {
                    tc_fence_after_sync();
                    const uint32_t sQ = smem_u32(tQ), sK = smem_u32(tK), sG = smem_u32(tG);
                    const uint32_t sP = smem_u32(tP), sdP = smem_u32(tdP);
                    issue<64, D, false, true, T / 16, C::CHT, C::CHT>(tmem + aQK, sdP, sK, true);             // + dP Kc
                    issue<64, D, true, true, T / 16, C::CHT, C::CHT>(tmem + aQK + kHi, sdP, sQ, true);        // + dP^T Qc
                    issue<64, D, true, true, T / 16, C::CHT, C::CHT>(tmem + aV + kHi, sP, sG, true);          // + P^T dO
                    issue_state_product<D>(tmem + aP, tQ, tG);                                                // Qc^T dO
                    mma_commit(barG1);
                }
                {
                    ok = wait_all(barG1, 1, a.status);
                    if (ok) {
                        tc_fence_after_sync();
                        if (tid == kIssuer && (u > 0 || tile > t0)) {
                            // every product has completed: fetch the next sub-chunk's zero-start state
                            const size_t nslot = u > 0 ? slot + (size_t)g.B * g.H * pl.ntile : (size_t)bh * pl.ntile + (tile - 1);
                            const char *src = reinterpret_cast<const char *>(a.slot_s + nslot * (D * D));
                            mbar_arrive_expect_tx(barS, (uint32_t)C::NCH * D * 16u);
                            for (int j = 0; j < C::NCH; ++j) bulk_g2s(tS + j * C::CHS, src + j * D * 16, D * 16, barS);
                        }
                        const bool inrow = r16 >= lo && r16 < hiv;
                        const size_t ro = (size_t)(my_off < 0 ? 0 : my_off);
#pragma unroll
                        for (int i = 0; i < L::NPC; ++i) {
                            const int jc = cg + L::NCG * i;
                            if (jc < C::NCH) {          // uniform over the warp
                                float a1[8], a2[8], x[8];
                                // lanes 0-15: dq accumulator and dO S_segment^T; lanes 16-31: dk and dv accumulators
                                tmem_ld8_pair(lane_base + tmem + aQK + 8 * jc, lane_base + tmem + aV + 8 * jc, a1, a2);
                                if (hf == 0) {
                                    float hh[8];
                                    ld8(vc.aux + 8 * jc, hh);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) a1[e] = fmaf(hh[e], a2[e], a1[e]);
                                } else if (inrow) {
                                    store_out8(dv + ro + 8 * jc, a2, a.accumulate != 0);
                                }
                                {
                                    // q*dq = Qc * (dq accumulator), k*dk = Kc * (dk accumulator): the decay factors cancel
                                    float t8[8];
                                    unpack_h8(*reinterpret_cast<const uint4 *>((hf ? tK : tQ) + jc * C::CHT + r16 * 16), t8);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) x[e] = t8[e] * a1[e];
                                }
#pragma unroll
                                for (int e = 0; e < 8; ++e) x[e] -= __shfl_xor_sync(0xffffffffu, x[e], 16);
                                {
                                    float lam[8], of[8];
                                    ld8(table + r16 * C::LAMP + 8 * jc, lam);
                                    ld8(vc.off + 8 * jc, of);
#pragma unroll
                                    for (int e = 0; e < 8; ++e) a1[e] *= ex2(hf ? of[e] - lam[e] : lam[e] - of[e]);
                                }
                                __syncwarp();           // both halves have read their gates before the table is overwritten
                                if (inrow) {
                                    if (hf == 0) st8(table + r16 * C::LAMP + 8 * jc, x);        // q*dq - k*dk
                                    store_out8((hf ? dk : dq) + ro + 8 * jc, a1, a.accumulate != 0);
                                }
                            }
                        }
                        // D <- 2^(2c) D + 2^c (Qc^T dO)
                        update_state<D, NT>(lane_base, tmem + aP, sm, Dst, vc.e2c, vc.ec);
                        if (u == 0 && tile > t0)
                            load_raw<D, NT, true, true, false, true>(raw, a.q, a.k, a.v, a.d_out, a.gate, rowOff + nxt * T);
                    }
                    tc_fence_before_sync();
                }
                par ^= 1;
            }
            // gate gradient of the tile: suffix sums of q*dq - k*dk down the rows plus what later tiles carry in
            SYNC_OR_DIE();
            {
                const bool active = tid < L::NSEG * D;
                const int seg = tid / D, c = tid - seg * D, r0 = seg * L::RPS;
                float sfx[L::RPS];
                if (active) {
                    float run = 0.f;
#pragma unroll
                    for (int j = L::RPS - 1; j >= 0; --j) {
                        if (r0 + j < nrow) run += table[(r0 + j) * C::LAMP + c];
                        sfx[j] = run;
                    }
                    sTot[seg * D + c] = run;
                }
                __syncthreads();
                if (active) {
                    float add = sCarry[cpar * D + c], all = 0.f;
#pragma unroll
                    for (int sgm = 0; sgm < L::NSEG; ++sgm) {
                        const float t = sTot[sgm * D + c];
                        if (sgm > seg) add += t;
                        all += t;
                    }
                    if (seg == 0) sCarry[(cpar ^ 1) * D + c] = sCarry[cpar * D + c] + all;
#pragma unroll
                    for (int j = 0; j < L::RPS; ++j) {
                        const int ro = r0 + j < nrow ? rowOff[cur * T + r0 + j] : -1;
                        if (ro >= 0) a.dgate[(size_t)ro + c] = (a.accumulate ? a.dgate[(size_t)ro + c] : 0.f) + (sfx[j] + add);
                    }
                }
                cpar ^= 1;
            }
            cur = nxt;
        }
    }
die:
    if (!ok && tid == kIssuer) mbar_wait(barS, par, a.status);      // let bulk copies in flight land
    cta_teardown(ctl, SM::tmem_cols);
}

#undef SYNC_OR_DIE

// ---- host side ----------------------------------------------------------------------------------
// Launch shapes per head size: worker threads per CTA and CTAs per SM of each kernel (the light
// kernels run more CTAs per SM on fewer registers, which hides the latency of their short tiles).
template <int D>
struct Shape {          // d = 64: two CTAs of 256 threads per SM
    static constexpr int NT_LOCAL_F = 256, NT_LOCAL_B = 256, NT_FWD = 256, NT_BWD = 256, OCC = 2;
};
template <>
struct Shape<72> {
    static constexpr int NT_LOCAL_F = 640, NT_LOCAL_B = 640, NT_FWD = 640, NT_BWD = 640, OCC = 1;
};

// A forward pass whose sequences are not cut (one segment each) runs the forward sweep alone, from the
// start state: no local sweep, no scan.  Cut sequences pay for the local sweep as well, about 0.7 of a
// forward sweep; the backward pass needs the local sweep (the per-tile states) in either case.
Plan make_plan(const Geom &g, int sms, int per_sm, bool backward)
{
    Plan p;
    p.ntile = (g.L + T - 1) / T;
    p.sub_max = g.C < T ? g.C : T;
    const long long slots = (long long)sms * per_sm, bh = (long long)g.B * g.H;
    long long best = -1;
    p.G = p.ntile;
    for (int G = p.ntile; G >= 1; --G) {
        const int nseg = (p.ntile + G - 1) / G;
        const long long rounds = (bh * nseg + slots - 1) / slots;
        long long cost = rounds * (G + 1) * 10;             // a segment costs about one tile of fill and drain
        if (!backward && nseg > 1) cost += cost * 7 / 10;
        if (best < 0 || cost < best) {
            best = cost;
            p.G = G;
        }
    }
    p.nseg = (p.ntile + p.G - 1) / p.G;
    return p;
}

struct SweepWs {
    float *seg_state, *seg_gamma, *seg_dstate, *seg_carry, *slot_g;
    __half *seg_state16, *slot_s;
    size_t bytes;
};
SweepWs carve(char *base, const Geom &g, const Plan &pl, bool backward)
{
    SweepWs w{};
    const size_t segs = (size_t)g.B * g.H * pl.nseg, dd = (size_t)g.dk * g.dv;
    size_t o = 0;
    auto take = [&](size_t bytes) { char *p = base + o; o += align256(bytes); return p; };
    w.seg_state = reinterpret_cast<float *>(take(segs * dd * 4));
    w.seg_gamma = reinterpret_cast<float *>(take(segs * g.dk * 4));
    if (backward) {
        const size_t slots = (size_t)kSlots * g.B * g.H * pl.ntile;
        w.seg_dstate = reinterpret_cast<float *>(take(segs * dd * 4));
        w.seg_carry = reinterpret_cast<float *>(take(segs * g.dk * 4));
        w.seg_state16 = reinterpret_cast<__half *>(take(segs * dd * 2));
        w.slot_s = reinterpret_cast<__half *>(take(slots * dd * 2));
        w.slot_g = reinterpret_cast<float *>(take(slots * g.dk * 4));
    }
    w.bytes = o;
    return w;
}

// CTAs per SM of the heaviest kernel of a pass: segments are sized for that many slots
int sweep_per_sm(int d, bool backward)
{
    (void)backward;
    return d == 64 ? Shape<64>::OCC : Shape<72>::OCC;
}

template <typename K>
dig_status set_smem(K kern, size_t bytes)
{
    return ensure_dynamic_smem(reinterpret_cast<const void *>(kern), bytes);
}

template <int D, bool BWD>
dig_status run(const GlaArgs &ga)
{
    using SH = Shape<D>;
    constexpr int NT_L = BWD ? SH::NT_LOCAL_B : SH::NT_LOCAL_F, NT_M = BWD ? SH::NT_BWD : SH::NT_FWD;
    constexpr int OCC_L = SH::OCC, OCC_M = SH::OCC;
    const Geom &g = ga.g;
    const int sms = device_sm_count();
    int *status = device_status_ptr();
    if (!status || sms <= 0) return DIG_ERR_CUDA;
    const Plan pl = make_plan(g, sms, OCC_M, BWD);
    const SweepWs w = carve(reinterpret_cast<char *>(ga.ws), g, pl, BWD);
    const long long total = (long long)g.B * g.H * pl.nseg;
    if (total > (1ll << 30) || (long long)g.B * g.L * g.H * D >= (1ll << 31)) return DIG_ERR_UNSUPPORTED;     // 31-bit row offsets
    SweepArgs a{};
    a.q = (const bf16 *)ga.q; a.k = (const bf16 *)ga.k; a.v = (const bf16 *)ga.v; a.d_out = (const bf16 *)ga.d_out;
    a.gate = ga.gate;
    a.out = ga.out; a.dq = ga.dq; a.dk = ga.dk; a.dv = ga.dv; a.dgate = ga.dgate;
    a.seg_state = w.seg_state; a.seg_gamma = w.seg_gamma; a.seg_dstate = w.seg_dstate; a.seg_carry = w.seg_carry;
    a.seg_state16 = w.seg_state16; a.slot_s = w.slot_s; a.slot_g = w.slot_g;
    a.status = status;
    a.accumulate = ga.accumulate;
    a.g = g;
    a.plan = pl;
    const int grid_l = (int)(total < (long long)sms * OCC_L ? total : (long long)sms * OCC_L);
    const int grid_m = (int)(total < (long long)sms * OCC_M ? total : (long long)sms * OCC_M);
    a.s_in = ga.sio.s_in;
    a.s_out = ga.sio.s_out;
    const bool sweep_only = !BWD && pl.nseg == 1;      // uncut sequences: the forward sweep starts from the start state itself
    dig_status st;
    // backward pass over uncut sequences whose start-state gradient is not asked for: the segment's own
    // contribution to the state gradient is never used, the local sweep only has to store the states
    const bool states_only = BWD && pl.nseg == 1 && ga.sio.ds_in == nullptr;
    if (states_only) {
        auto kern = sweep_local<D, SH::NT_LOCAL_F, false, OCC_L, true>;
        constexpr size_t smem = LocalSmem<D, SH::NT_LOCAL_F, false>::bytes;
        if ((st = set_smem(kern, smem)) != DIG_OK) return st;
        KernelTimer t(KID_SW_LOCAL, ga.stream);
        launch_pdl(kern, dim3(grid_l), dim3(SH::NT_LOCAL_F), smem, ga.stream, a);
        if ((st = cuda_ok(cudaGetLastError())) != DIG_OK) return st;
    } else if (!sweep_only) {
        auto kern = sweep_local<D, NT_L, BWD, OCC_L>;
        constexpr size_t smem = LocalSmem<D, NT_L, BWD>::bytes;
        if ((st = set_smem(kern, smem)) != DIG_OK) return st;
        KernelTimer t(KID_SW_LOCAL, ga.stream);
        launch_pdl(kern, dim3(grid_l), dim3(NT_L), smem, ga.stream, a);
        if ((st = cuda_ok(cudaGetLastError())) != DIG_OK) return st;
    }
    if (!sweep_only) {
        auto kern = seg_scan<D, BWD>;
        KernelTimer t(KID_SW_SCAN, ga.stream);
        launch_pdl(kern, dim3(g.B * g.H, D / 8), dim3(64), 0, ga.stream, w.seg_state, (const float *)w.seg_gamma, w.seg_dstate,
                   w.seg_carry, w.seg_state16, ga.sio.s_in, ga.sio.s_out, ga.sio.ds_out, ga.sio.ds_in, pl.nseg);
        if ((st = cuda_ok(cudaGetLastError())) != DIG_OK) return st;
    }
    const bool f32 = ga.dtype == DIG_BF16_F32OUT;
    if constexpr (!BWD) {
        constexpr size_t smem = FwdSmem<D, NT_M>::bytes;
        auto k16 = sweep_fwd<D, NT_M, bf16, OCC_M>;
        auto k32 = sweep_fwd<D, NT_M, float, OCC_M>;
        if ((st = set_smem(k16, smem)) != DIG_OK || (st = set_smem(k32, smem)) != DIG_OK) return st;
        KernelTimer t(KID_SW_FWD, ga.stream);
        launch_pdl(f32 ? k32 : k16, dim3(grid_m), dim3(NT_M), smem, ga.stream, a);
    } else {
        constexpr size_t smem = BwdSmem<D, NT_M>::bytes;
        auto k16 = sweep_bwd<D, NT_M, bf16, OCC_M>;
        auto k32 = sweep_bwd<D, NT_M, float, OCC_M>;
        if ((st = set_smem(k16, smem)) != DIG_OK || (st = set_smem(k32, smem)) != DIG_OK) return st;
        KernelTimer t(KID_SW_BWD, ga.stream);
        launch_pdl(f32 ? k32 : k16, dim3(grid_m), dim3(NT_M), smem, ga.stream, a);
    }
    return cuda_ok(cudaGetLastError());
}

}  // namespace

bool sweep_supports(int dk, int dv, int chunk, int dtype)
{
    if (dtype != DIG_BF16 && dtype != DIG_BF16_F32OUT) return false;
    (void)chunk;                     // every chunk size is worked in 64-token tiles, shorter ones as sub-chunks
    return dk == dv && (dk == 64 || dk == 72);
}

size_t sweep_workspace_bytes(const Geom &g, bool backward)
{
    int sms = device_sm_count();
    if (sms <= 0) sms = 148;
    const Plan pl = make_plan(g, sms, sweep_per_sm(g.dk, backward), backward);
    return carve(nullptr, g, pl, backward).bytes;
}

namespace {

// fp32 sums -> bf16 results (round to nearest even), 8 elements per thread.
__global__ void __launch_bounds__(256) round_to_bf16(const float *__restrict__ src, bf16 *__restrict__ dst, size_t n8)
{
    pdl_wait();
    pdl_launch_dependents();
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= n8) return;
    float f[8];
    ld8(src + 8 * i, f);
    store_out8(dst + 8 * i, f);
}
dig_status launch_round(const float *src, void *dst, size_t n, cudaStream_t s)
{
    const size_t n8 = n / 8;
    launch_pdl(round_to_bf16, dim3((unsigned)((n8 + 255) / 256)), dim3(256), 0, s, src, (bf16 *)dst, n8);
    return cuda_ok(cudaGetLastError());
}

}  // namespace

// Several scan orders summed (Algorithm 2 / Algorithm 3): the orders run one after the other, each
// adding its fp32 results to the same buffers, which are rounded to the storage type once at the end.
size_t sweep_multi_workspace_bytes(const Geom &g, bool backward, int dtype)
{
    size_t n = align256(sweep_workspace_bytes(g, backward));
    if (dtype == DIG_BF16) {
        const size_t tok = (size_t)g.B * g.L * g.H;
        n += backward ? align256(tok * g.dk * 4) * 2 + align256(tok * g.dv * 4) : align256(tok * g.dv * 4);
    }
    return n;
}

dig_status sweep_gla_fwd_multi(const GlaArgs &a0, unsigned mask)
{
    GlaArgs a = a0;
    const size_t tok = (size_t)a.g.B * a.g.L * a.g.H;
    char *extra = reinterpret_cast<char *>(a0.ws) + align256(sweep_workspace_bytes(a.g, false));
    const bool narrow = a0.dtype == DIG_BF16;
    a.dtype = DIG_BF16_F32OUT;
    if (narrow) a.out = extra;
    bool first = true;
    for (int d = 0; d < 4; ++d) {
        if (!(mask >> d & 1)) continue;
        a.g.dir = d;
        a.accumulate = first ? 0 : 1;
        first = false;
        const dig_status st = sweep_gla_fwd(a);
        if (st != DIG_OK) return st;
    }
    return narrow ? launch_round(reinterpret_cast<const float *>(extra), a0.out, tok * a.g.dv, a.stream) : DIG_OK;
}

dig_status sweep_gla_bwd_multi(const GlaArgs &a0, unsigned mask)
{
    GlaArgs a = a0;
    const size_t tok = (size_t)a.g.B * a.g.L * a.g.H;
    char *extra = reinterpret_cast<char *>(a0.ws) + align256(sweep_workspace_bytes(a.g, true));
    const bool narrow = a0.dtype == DIG_BF16;
    a.dtype = DIG_BF16_F32OUT;
    float *sq = reinterpret_cast<float *>(extra), *sk = reinterpret_cast<float *>(extra + align256(tok * a.g.dk * 4));
    float *sv = reinterpret_cast<float *>(extra + 2 * align256(tok * a.g.dk * 4));
    if (narrow) { a.dq = sq; a.dk = sk; a.dv = sv; }
    bool first = true;
    for (int d = 0; d < 4; ++d) {
        if (!(mask >> d & 1)) continue;
        a.g.dir = d;
        a.accumulate = first ? 0 : 1;
        first = false;
        const dig_status st = sweep_gla_bwd(a);
        if (st != DIG_OK) return st;
    }
    if (!narrow) return DIG_OK;
    dig_status st;
    if ((st = launch_round(sq, a0.dq, tok * a.g.dk, a.stream)) != DIG_OK) return st;
    if ((st = launch_round(sk, a0.dk, tok * a.g.dk, a.stream)) != DIG_OK) return st;
    return launch_round(sv, a0.dv, tok * a.g.dv, a.stream);
}

dig_status sweep_gla_fwd(const GlaArgs &a)
{
    return a.g.dk == 64 ? run<64, false>(a) : run<72, false>(a);
}
dig_status sweep_gla_bwd(const GlaArgs &a)
{
    return a.g.dk == 64 ? run<64, true>(a) : run<72, true>(a);
}

}  // namespace dig
