// Building blocks of the tcgen05 "sweep" kernels for chunkwise gated linear attention (Eq. attn_gla
// evaluated chunk by chunk, Section 3.5).  A CTA walks over consecutive 64-token tiles of one
// (batch, head) sequence and keeps the d_k x d_v state of the recurrence in registers, so per-chunk
// states never travel through memory in the forward pass.
//
// Operand tiles are fp16 (11 significant bits, like tf32, at half the bytes and with one copy
// serving both operand orientations).  fp16's narrow exponent is handled by centring the in-chunk
// decay: with Lam the cumulative gate inside a (sub-)chunk and c = Lam_end / 2 per channel, the
// tiles hold q*exp(Lam - c) and k*exp(c - Lam), whose factors stay within exp(+-|Lam_end|/2).  A
// tile whose gates sum to more than kSubLimit is worked in shorter sub-chunks (32, 16 or 8 rows of
// the same tile, the other rows zero), each with its own centring; conversions saturate instead of
// overflowing.
//
// Tile layout: no swizzle, "chunk-major": element (row, col) of a tile with R rows sits at
//   (col / 8) * (16 R + 16) + 16 row + 2 (col % 8)
// i.e. 8-column chunks of 16 bytes per row, rows contiguous within a chunk, one 16-byte pad per
// chunk.  Every 8 x 16-byte core matrix is contiguous, which is what the non-swizzled tcgen05
// matrix descriptors want in both orientations, any number of columns that is a multiple of 8
// works, and both a warp that stores 32 rows of one chunk and a warp that stores the chunks of 4
// rows touch 32 different banks.
#pragma once

#include <cuda_fp16.h>

#include "dig_common.cuh"
#include "umma.cuh"

namespace dig {
namespace sw {

using namespace umma;
using bf16 = __nv_bfloat16;

constexpr int T = 64;                       // rows (scan positions) of a tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kSubLimit = 23.0f;          // largest |sum of gates| (log2 units, = 15.9 nats) of one (sub-)chunk
constexpr int kMinSub = 8;                  // shortest sub-chunk
constexpr int kSlots = T / kMinSub;         // sub-chunks a tile can have
constexpr int kStatusTimeout = 1, kStatusRange = 2;

template <int D>
struct Cfg {
    static_assert(D % 8 == 0 && D >= 16 && D <= 128, "head size");
    static constexpr int NCH = D / 8;               // 8-column chunks that hold data
    static constexpr int KS = (D + 15) / 16;        // MMA steps of a contraction over the channels
    static constexpr int NCHP = 2 * KS;             // chunks a tile provides (a last zero chunk pads odd counts)
    static constexpr int RS = 16 * KS;              // rows of a state tile (zero rows beyond D)
    static constexpr bool BIGM = D > 64;            // products with channels along M run as M = 128
    static constexpr int NACC = BIGM ? RS : D;      // accumulator columns of a product with channels along N
    static constexpr int CHT = T * 16 + 16;         // chunk stride of a token tile (64 rows)
    static constexpr int CHS = RS * 16 + 16;        // chunk stride of a state tile (RS rows)
    static constexpr int TILE_T = NCHP * CHT, TILE_S = NCHP * CHS, TILE_P = (T / 8) * CHT;
    static constexpr int LAMP = D + 4;              // floats per row of the gate table
    static_assert(BIGM || (NCH % 2 == 0), "heads of at most 64 channels split their state products in two halves");
};

// Work split of a CTA of NT threads (lane 0 of the last warp also issues the MMAs and the bulk copies).
template <int D, int NT>
struct Lay {
    using C = Cfg<D>;
    static_assert(NT % 128 == 0, "four warps per tensor-memory lane quarter group");
    static constexpr int NCG = NT / 128;                          // column groups: warps that share a lane quarter
    static constexpr int NSEG = NT / D;                           // row segments of the column scans
    static constexpr int RPS = (T + NSEG - 1) / NSEG;             // rows per segment
    static constexpr int NIT = (T * C::NCH + NT - 1) / NT;        // (row, chunk) items per thread of one tensor
    static constexpr int NPC = (C::NCH + NCG - 1) / NCG;          // channel chunks per thread in row-wise epilogues
    static constexpr int NPT = (T / 8 + NCG - 1) / NCG;           // token-column chunks per thread of a score tile
    static constexpr int HCH = C::NCH / 2;                        // chunks per half (state products of small heads)
    static constexpr int NPS = C::BIGM ? NPC : (HCH + NCG - 1) / NCG;   // state chunks per thread
    static_assert(NSEG >= 1, "thread count");
};

struct Plan {
    int ntile;      // 64-token tiles per sequence
    int nseg;       // segments per sequence (one CTA sweeps one segment)
    int G;          // tiles per segment
    int sub_max;    // longest sub-chunk allowed (the requested chunk size, at most 64)
};

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two floats -> packed fp16 (first argument in the low half), round to nearest, saturating to the
// largest finite value instead of overflowing to infinity.
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint4 pack_h8(const float (&f)[8])
{
    return make_uint4(pack_h2(f[0], f[1]), pack_h2(f[2], f[3]), pack_h2(f[4], f[5]), pack_h2(f[6], f[7]));
}
__device__ __forceinline__ void unpack_h8(const uint4 &u, float (&f)[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 v = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
        f[2 * i] = v.x;
        f[2 * i + 1] = v.y;
    }
}
__device__ __forceinline__ void unpack_b8(const uint4 &u, float (&f)[8])
{
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void ld8(const float *p, float (&f)[8])
{
    const float4 a = *reinterpret_cast<const float4 *>(p), b = *reinterpret_cast<const float4 *>(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}
__device__ __forceinline__ void st8(float *p, const float (&f)[8])
{
    *reinterpret_cast<float4 *>(p) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4 *>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
}
// 8 results to global memory in the output storage type.  `add`: on top of what is there (fp32
// outputs only; used when several scan orders are summed into one buffer).
__device__ __forceinline__ void store_out8(float *p, const float (&f)[8], bool add = false)
{
    if (add) {
        float o[8];
        ld8(p, o);
#pragma unroll
        for (int e = 0; e < 8; ++e) o[e] += f[e];
        st8(p, o);
    } else {
        st8(p, f);
    }
}
__device__ __forceinline__ void store_out8(bf16 *p, const float (&f)[8], bool = false)
{
    uint4 u;
    __nv_bfloat162 t;
    t = __floats2bfloat162_rn(f[0], f[1]); u.x = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[2], f[3]); u.y = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[4], f[5]); u.z = *reinterpret_cast<uint32_t *>(&t);
    t = __floats2bfloat162_rn(f[6], f[7]); u.w = *reinterpret_cast<uint32_t *>(&t);
    *reinterpret_cast<uint4 *>(p) = u;
}

// ---- matrix descriptors of chunk-major tiles -----------------------------------------------------
// K-major view (tile rows = M or N index, contraction along the columns): the two 8-column chunks
// of a 16-wide step are `ch` bytes apart (leading offset), 8-row groups 128 bytes (stride offset).
// MN-major view (tile rows = contraction index, columns = M or N index): 8-row groups along the
// contraction 128 bytes apart (leading offset), 8-column chunks along M / N `ch` bytes (stride).
__device__ __forceinline__ uint64_t kdesc(uint32_t saddr, uint32_t ch) { return make_desc(saddr, ch, 128, 0); }
__device__ __forceinline__ uint64_t mdesc(uint32_t saddr, uint32_t ch) { return make_desc(saddr, 128, ch, 0); }

// D[tmem] (+)= A * B over KSTEPS steps of 16 along the contraction.  a / b: shared-memory address
// of the first element the product uses (a row or chunk offset selects a slice), ach / bch: chunk
// strides of the tiles (compile-time, so every descriptor is the first one plus a constant in its
// low word: shared-memory addresses stay below 2^18, the address field cannot carry into the next).
template <int M, int N, bool A_MN, bool B_MN, int KSTEPS, uint32_t ACH, uint32_t BCH>
__device__ __forceinline__ void issue(uint32_t d_tmem, uint32_t a, uint32_t b, bool accumulate)
{
    static_assert((M == 64 && N % 8 == 0) || (M == 128 && N % 16 == 0), "instruction shape");
    constexpr uint32_t idesc = idesc_f16(M, N, A_MN, B_MN);
    const uint64_t da = A_MN ? mdesc(a, ACH) : kdesc(a, ACH), db = B_MN ? mdesc(b, BCH) : kdesc(b, BCH);
    constexpr uint32_t sa = A_MN ? 16u : (2u * ACH) >> 4, sb = B_MN ? 16u : (2u * BCH) >> 4;
    const uint32_t alo = (uint32_t)da, ahi = (uint32_t)(da >> 32), blo = (uint32_t)db, bhi = (uint32_t)(db >> 32);
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
        const uint64_t xa = ((uint64_t)ahi << 32) | (alo + kk * sa), xb = ((uint64_t)bhi << 32) | (blo + kk * sb);
        mma_f16(d_tmem, xa, xb, idesc, accumulate || kk > 0);
    }
}

struct Ctl {
    uint64_t bar[4];
    uint32_t tmem_base;
    uint32_t pad;
};

// Element offset of the (batch b, head h) row of the token at scan position 64*tile + row in a
// [B][L][H][D] tensor, or -1 past the end of the sequence (the host checks that offsets fit 31 bits).
__device__ __forceinline__ int tile_row_offset(const Geom &g, int b, int h, int d, int tile, int row)
{
    const int p = tile * T + row;
    return p < g.L ? (int)tok_offset(g, b, scan_token(p, g.dir, g.gh, g.gw, g.L), h, d) : -1;
}

// ---- rows of q, k, v, dO and the gates of one tile, prefetched into registers ------------------
template <int NIT, bool HQ, bool HD>
struct Raw {
    uint4 k[NIT], v[NIT], q[HQ ? NIT : 1], d[HD ? NIT : 1];
    float4 g0[NIT], g1[NIT];
};
__device__ __forceinline__ uint4 ldg16(const bf16 *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
__device__ __forceinline__ float4 ldg16(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

// Item i of a thread is (row, chunk) = divmod(tid + NT*i, NCH): consecutive threads read consecutive
// 16-byte pieces of a token row.  Rows past the end of the sequence read the tensor's first row (masked later).
// GATES / ROWS: which part to load (the gates are needed first, the bf16 rows can follow later).
template <int D, int NT>
__device__ __forceinline__ bool item_exists(int it)
{
    return (T * Cfg<D>::NCH) % NT == 0 || it < T * Cfg<D>::NCH;     // every thread has all its items when NT divides the count
}
template <int D, int NT, bool HQ, bool HD, bool GATES = true, bool ROWS = true>
__device__ __forceinline__ void load_raw(Raw<Lay<D, NT>::NIT, HQ, HD> &r, const bf16 *q, const bf16 *k, const bf16 *v,
                                         const bf16 *d_out, const float *gate, const int *row_off)
{
    constexpr int NCH = Cfg<D>::NCH;
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NIT; ++i) {
        const int it = (int)threadIdx.x + NT * i;
        if (item_exists<D, NT>(it)) {
            const int row = it / NCH, j = it - row * NCH;
            const int ro = row_off[row];
            const uint32_t off = (uint32_t)(ro < 0 ? 0 : ro) + 8u * j;
            if (ROWS) {
                r.k[i] = ldg16(k + off);
                r.v[i] = ldg16(v + off);
                if (HQ) r.q[i] = ldg16(q + off);
                if (HD) r.d[i] = ldg16(d_out + off);
            }
            if (GATES) {
                r.g0[i] = ldg16(gate + off);
                r.g1[i] = ldg16(gate + off + 4);
            }
        }
    }
}

// Asks the L2 for one token row of every input tensor (a tile further ahead than the register
// prefetch reaches, so that the register loads find their lines in the L2).
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" :: "l"(p)); }
template <int D, bool HQ, bool HD>
__device__ __forceinline__ void prefetch_row(const bf16 *q, const bf16 *k, const bf16 *v, const bf16 *d_out,
                                             const float *gate, int row_off)
{
    if (row_off < 0) return;
#pragma unroll
    for (int b = 0; b < 2 * D; b += 128) {
        const int e = (b < 2 * D - 16 ? b : 2 * D - 16) / 2;        // the last piece covers the row's end
        prefetch_l2(k + row_off + e);
        prefetch_l2(v + row_off + e);
        if (HQ) prefetch_l2(q + row_off + e);
        if (HD) prefetch_l2(d_out + row_off + e);
    }
    prefetch_l2(k + row_off + D - 8);
    prefetch_l2(v + row_off + D - 8);
    if (HQ) prefetch_l2(q + row_off + D - 8);
    if (HD) prefetch_l2(d_out + row_off + D - 8);
#pragma unroll
    for (int b = 0; b < 4 * D; b += 128) prefetch_l2(gate + row_off + b / 4);
    prefetch_l2(gate + row_off + D - 4);
}

// Gates of the prefetched tile into the table, in log2 units, zero for rows past the end.
template <int D, int NT, bool HQ, bool HD>
__device__ __forceinline__ void write_gates(const Raw<Lay<D, NT>::NIT, HQ, HD> &r, float *table, const int *row_off)
{
    constexpr int NCH = Cfg<D>::NCH, LAMP = Cfg<D>::LAMP;
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NIT; ++i) {
        const int it = (int)threadIdx.x + NT * i;
        if (item_exists<D, NT>(it)) {
            const int row = it / NCH, j = it - row * NCH;
            const float sc = row_off[row] >= 0 ? kLog2e : 0.f;
            float *dst = table + row * LAMP + 8 * j;
            *reinterpret_cast<float4 *>(dst) = make_float4(r.g0[i].x * sc, r.g0[i].y * sc, r.g0[i].z * sc, r.g0[i].w * sc);
            *reinterpret_cast<float4 *>(dst + 4) = make_float4(r.g1[i].x * sc, r.g1[i].y * sc, r.g1[i].z * sc, r.g1[i].w * sc);
        }
    }
}

// Per-channel vectors of one (sub-)chunk, double-buffered by iteration parity:
//   off = base + c   (gate prefix at the sub-chunk's start plus half its total: exponent offset of the tiles)
//   ec  = 2^c, e2c = 2^(2c) (the sub-chunk's total decay), aux = kernel specific
struct Vec {
    float *off, *ec, *e2c, *aux;
};
template <int D>
__device__ __forceinline__ Vec vec_of(float *base, int parity)
{
    float *p = base + parity * 4 * D;
    return Vec{p, p + D, p + 2 * D, p + 3 * D};
}

// Turns the table's rows into inclusive prefix sums down the rows (all NT threads).  Returns, uniformly, whether some channel's total
// over the tile exceeds kSubLimit in magnitude.  tot_out (threads < D): the channel's total.
// Contains two barriers; the caller must have placed one after write_gates.  on_total(c, total) runs
// in the thread that owns channel c before the last barrier: what it writes to shared memory is
// visible to everyone afterwards (the kernels put the vectors of an undivided tile there, which saves
// them a barrier of their own).
template <int D, int NT, typename F>
__device__ __forceinline__ bool gate_prefix(float *table, float *sTot, float &tot_out, F on_total)
{
    using L = Lay<D, NT>;
    constexpr int LAMP = Cfg<D>::LAMP;
    const int tid = threadIdx.x;
    const bool active = tid < L::NSEG * D;
    const int seg = tid / D, c = tid - seg * D, r0 = seg * L::RPS;
    float a[L::RPS];
    if (active) {
        float run = 0.f;
#pragma unroll
        for (int j = 0; j < L::RPS; ++j) {
            if (r0 + j < T) run += table[(r0 + j) * LAMP + c];
            a[j] = run;
        }
        sTot[seg * D + c] = run;
    }
    __syncthreads();
    bool big = false;
    if (active) {
        float add = 0.f, tot = 0.f;
#pragma unroll
        for (int s = 0; s < L::NSEG; ++s) {
            const float t = sTot[s * D + c];
            if (s < seg) add += t;
            tot += t;
        }
#pragma unroll
        for (int j = 0; j < L::RPS; ++j)
            if (r0 + j < T) table[(r0 + j) * LAMP + c] = a[j] + add;
        tot_out = tot;
        big = seg == 0 && fabsf(tot) > kSubLimit;
        if (seg == 0) on_total(c, tot);
    }
    return __syncthreads_or(big) != 0;
}

// Longest sub-chunk length (a power of two between kMinSub and `start`) for which every aligned
// window of the tile keeps |sum of gates| <= kSubLimit; kMinSub if none does (then *range_bad is set).
// Uniform result; contains barriers (all threads of the CTA must call it).
template <int D>
__device__ __forceinline__ int choose_sub(const float *table, int start, bool *range_bad)
{
    constexpr int LAMP = Cfg<D>::LAMP;
    const int c = threadIdx.x;
    int s = start;
    for (;;) {
        bool viol = false;
        if (c < D) {
            float prev = 0.f;
            for (int end = s; end <= T; end += s) {
                const float cur = table[(end - 1) * LAMP + c];
                viol |= fabsf(cur - prev) > kSubLimit;
                prev = cur;
            }
        }
        viol = __syncthreads_or(viol) != 0;
        if (!viol) { *range_bad = false; return s; }
        if (s <= kMinSub) { *range_bad = true; return s; }
        s >>= 1;
    }
}

// Thread -> rows and chunks -------------------------------------------------------------------
// Row-wise work on accumulators of token rows (M = 64): the thread's row is 16*quarter + lane % 16;
// lanes 16-31 see the second accumulator that shares the columns.  Its channel chunks are
// cg, cg + NCG, ...  State work (accumulator rows = key channels): for heads of at most 64 channels
// the product is split into two value-column halves that share columns the same way (row = same
// formula, half = lane / 16); for larger heads the product has M = 128 and the row is
// 32*quarter + lane.
template <int D, int NT>
struct StateMap {
    using C = Cfg<D>;
    using L = Lay<D, NT>;
    int c;          // key channel (row of the state)
    bool valid;
    int cg, hf;
    __device__ __forceinline__ StateMap()
    {
        const int tid = threadIdx.x, lane = tid & 31, q4 = (tid >> 5) & 3;
        cg = tid >> 7;
        hf = lane >> 4;
        c = C::BIGM ? 32 * q4 + lane : 16 * q4 + (lane & 15);
        valid = c < D;
    }
    // value-column chunk of piece i, and whether the piece exists (uniform over the warp)
    __device__ __forceinline__ bool has(int i) const { return cg + L::NCG * i < (C::BIGM ? C::NCH : L::HCH); }
    __device__ __forceinline__ int echunk(int i) const { return (C::BIGM ? 0 : hf * L::HCH) + cg + L::NCG * i; }
    __device__ __forceinline__ uint32_t tcol(int i) const { return 8u * (uint32_t)(cg + L::NCG * i); }
};

// state (fp32 registers) -> fp16 state tile, rows scaled by ec (= 2^c of the consuming sub-chunk)
template <int D, int NT>
__device__ __forceinline__ void write_state_tile(char *tile, const StateMap<D, NT> &m, const float (&S)[Lay<D, NT>::NPS][8],
                                                 const float *ec)
{
    if (!m.valid) return;
    const float f = ec[m.c];
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NPS; ++i)
        if (m.has(i)) {
            float x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = S[i][e] * f;
            *reinterpret_cast<uint4 *>(tile + m.echunk(i) * Cfg<D>::CHS + m.c * 16) = pack_h8(x);
        }
}
// the same values to a dense [NCH][D][8] fp16 slot in global memory
template <int D, int NT>
__device__ __forceinline__ void write_state_slot(__half *slot, const StateMap<D, NT> &m, const float (&S)[Lay<D, NT>::NPS][8],
                                                 const float *ec)
{
    if (!m.valid) return;
    const float f = ec[m.c];
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NPS; ++i)
        if (m.has(i)) {
            float x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] = S[i][e] * f;
            *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(slot) + (m.echunk(i) * D + m.c) * 16) = pack_h8(x);
        }
}
// S <- e2c * S + ec * U, U read from the accumulator at tensor-memory column `acc`
template <int D, int NT>
__device__ __forceinline__ void update_state(uint32_t tmem_lane_base, uint32_t acc, const StateMap<D, NT> &m,
                                             float (&S)[Lay<D, NT>::NPS][8], const float *decay, const float *scale)
{
    const float fd = m.valid ? decay[m.c] : 0.f, fs = m.valid ? scale[m.c] : 0.f;
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NPS; ++i)
        if (m.has(i)) {          // uniform over the warp: tcgen05.ld is a warp-wide instruction
            float u[8];
            tmem_ld8(tmem_lane_base + acc + m.tcol(i), u);
#pragma unroll
            for (int e = 0; e < 8; ++e) S[i][e] = fd * S[i][e] + fs * u[e];
        }
}
template <int D, int NT>
__device__ __forceinline__ void load_state(const float *src, const StateMap<D, NT> &m, float (&S)[Lay<D, NT>::NPS][8])
{
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NPS; ++i) {
        if (m.has(i) && m.valid && src) ld8(src + (size_t)m.c * D + 8 * m.echunk(i), S[i]);
        else {
#pragma unroll
            for (int e = 0; e < 8; ++e) S[i][e] = 0.f;
        }
    }
}
template <int D, int NT>
__device__ __forceinline__ void store_state(float *dst, const StateMap<D, NT> &m, const float (&S)[Lay<D, NT>::NPS][8])
{
    if (!m.valid) return;
#pragma unroll
    for (int i = 0; i < Lay<D, NT>::NPS; ++i)
        if (m.has(i)) st8(dst + (size_t)m.c * D + 8 * m.echunk(i), S[i]);
}

// Zero-fills n16 16-byte words of shared memory with the CTA's threads.
__device__ __forceinline__ void zero_smem(char *p, int bytes)
{
    for (int i = threadIdx.x * 16; i < bytes; i += blockDim.x * 16) *reinterpret_cast<uint4 *>(p + i) = make_uint4(0, 0, 0, 0);
}

}  // namespace sw

// Host side of the sweep family (gla_sweep.cu).
bool sweep_supports(int dk, int dv, int chunk, int dtype);
size_t sweep_workspace_bytes(const Geom &g, bool backward);
dig_status sweep_gla_fwd(const GlaArgs &a);
dig_status sweep_gla_bwd(const GlaArgs &a);
// Sums over the scan orders of `mask` (bit d = direction d); outputs in the storage type of a.dtype.
size_t sweep_multi_workspace_bytes(const Geom &g, bool backward, int dtype);
dig_status sweep_gla_fwd_multi(const GlaArgs &a, unsigned mask);
dig_status sweep_gla_bwd_multi(const GlaArgs &a, unsigned mask);

}  // namespace dig
