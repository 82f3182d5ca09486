// Building blocks shared by the tensor-core GLA kernels: work-item decoding, coalesced row
// loads, conversion to tf32 and stores into the two swizzled operand-tile formats of umma.cuh,
// the in-chunk cumulative gate table, and lean tcgen05.mma issue loops.
#pragma once

#include "dig_common.cuh"
#include "umma.cuh"

namespace dig {
namespace tc {

using namespace umma;
using bf16 = __nv_bfloat16;

constexpr int T = 64;                    // tokens per chunk tile
constexpr int DK = 64, DV = 64;          // head sizes served by this family
constexpr int kLamPitch = 68;            // floats per row of the gate table (conflict-free 16-byte reads)
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One chunk of one (batch, head) sequence; `id` runs over all chunks of the call.
struct Item {
    int b, h, chunk;
    bool valid;
};
__device__ __forceinline__ Item item_of(const Geom &g, int id, int total)
{
    Item it;
    it.valid = id < total;
    const int bh = it.valid ? id / g.N : 0;
    it.chunk = it.valid ? id - bh * g.N : 0;
    it.b = bh / g.H;
    it.h = bh - it.b * g.H;
    return it;
}
// One of two items without indexing an array (keeps both in registers).
__device__ __forceinline__ Item pick(const Item &a, const Item &b, bool second)
{
    Item it;
    it.b = second ? b.b : a.b;
    it.h = second ? b.h : a.h;
    it.chunk = second ? b.chunk : a.chunk;
    it.valid = second ? b.valid : a.valid;
    return it;
}
// Canonical token of tile row r of the item, or -1 for rows past the end of the sequence.
__device__ __forceinline__ int item_token(const Geom &g, const Item &it, int r)
{
    const int p = it.chunk * T + r;
    return (it.valid && p < g.L) ? scan_token(p, g.dir, g.gh, g.gw, g.L) : -1;
}

// Element offset of tile row r of the item in a [B][L][H][64] tensor; rows past the end of the
// sequence map to token 0 (loads stay unconditional, the consumer zeroes the values).
__device__ __forceinline__ size_t row_offset(const Geom &g, const Item &it, int r)
{
    const int tok = item_token(g, it, r);
    return tok_offset(g, it.b, tok < 0 ? 0 : tok, it.h, 64);
}
__device__ __forceinline__ uint4 ldg16(const bf16 *p) { return __ldg(reinterpret_cast<const uint4 *>(p)); }
__device__ __forceinline__ float4 ldg16(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

// `keep` = false turns the row into zeros.
// `flip`: the lanes that hold columns 32-63 of a row keep the two 4-column halves of their 8 columns
// exchanged in registers (f[0..3] = columns col8+4..col8+7) and store the upper half first.  The 8
// lanes that serve one 16-byte store phase then hit 8 different bank groups of an operand tile or of
// the gate table; in natural order lane j and lane j+4 collide.  The tile stores, the gate loads and
// read_lam8 take the same flag, so the exchange costs four selects per input vector and nothing else.
__device__ __forceinline__ void unpack8(const uint4 &u, float (&f)[8], bool keep = true, bool flip = false)
{
    const uint32_t m = keep ? 0xffffffffu : 0u;
    const uint32_t w[4] = {(flip ? u.z : u.x) & m, (flip ? u.w : u.y) & m, (flip ? u.x : u.z) & m, (flip ? u.y : u.w) & m};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ float4 tf32x4(float a, float b, float c, float d)
{
    return make_float4(to_tf32(a), to_tf32(b), to_tf32(c), to_tf32(d));
}

// ---- stores into operand tiles (ROWS rows, column blocks of 32 words) -----------------------
// 8 consecutive columns starting at col8 (a multiple of 8).
// ROUND = false is for values that are exact in tf32 already (bf16 numbers, or rounded before).
template <int ROWS, bool ROUND = true>
__device__ __forceinline__ void st_k8(char *tile, int row, int col8, const float (&f)[8], bool flip)
{
    char *base = tile + (col8 >> 5) * (ROWS * 128) + row * 128;
    const int c = (col8 & 31) >> 2, s = row & 7;
    const float4 lo = ROUND ? tf32x4(f[0], f[1], f[2], f[3]) : make_float4(f[0], f[1], f[2], f[3]);
    const float4 hi = ROUND ? tf32x4(f[4], f[5], f[6], f[7]) : make_float4(f[4], f[5], f[6], f[7]);
    const int fl = flip ? 1 : 0;          // f[0..3] belong to piece c + fl (see unpack8)
    float4 *p0 = reinterpret_cast<float4 *>(base + (((c + fl) ^ s) << 4));
    float4 *p1 = reinterpret_cast<float4 *>(base + (((c + 1 - fl) ^ s) << 4));
    *p0 = lo;
    *p1 = hi;
}
template <int ROWS, bool ROUND = true>
__device__ __forceinline__ void st_m8(char *tile, int row, int col8, const float (&f)[8], bool flip)
{
    char *base = tile + (col8 >> 5) * (ROWS * 128) + row * 128 + (((((col8 & 31) >> 3)) ^ (row & 3)) << 5);
    const float4 lo = ROUND ? tf32x4(f[0], f[1], f[2], f[3]) : make_float4(f[0], f[1], f[2], f[3]);
    const float4 hi = ROUND ? tf32x4(f[4], f[5], f[6], f[7]) : make_float4(f[4], f[5], f[6], f[7]);
    const int fl = flip ? 16 : 0;         // f[0..3] belong to the upper 16 bytes of the atom in flipped lanes
    float4 *p0 = reinterpret_cast<float4 *>(base + fl), *p1 = reinterpret_cast<float4 *>(base + 16 - fl);
    *p0 = lo;
    *p1 = hi;
}
// 4 consecutive columns starting at col4 (a multiple of 4), rounded to tf32 unless ROUND = false.
template <int ROWS, bool ROUND = true>
__device__ __forceinline__ void st_k4(char *tile, int row, int col4, float4 v)
{
    *reinterpret_cast<float4 *>(tile + (col4 >> 5) * (ROWS * 128) + row * 128 + ((((col4 & 31) >> 2) ^ (row & 7)) << 4)) =
        ROUND ? tf32x4(v.x, v.y, v.z, v.w) : v;
}
template <int ROWS, bool ROUND = true>
__device__ __forceinline__ void st_m4(char *tile, int row, int col4, float4 v)
{
    *reinterpret_cast<float4 *>(tile + (col4 >> 5) * (ROWS * 128) + row * 128 +
                                (((((col4 & 31) >> 3)) ^ (row & 3)) << 5) + ((col4 & 4) << 2)) =
        ROUND ? tf32x4(v.x, v.y, v.z, v.w) : v;
}
// 8 consecutive columns of an M-format tile back into registers.
template <int ROWS>
__device__ __forceinline__ void ld_m8(const char *tile, int row, int col8, float (&f)[8])
{
    const char *base = tile + (col8 >> 5) * (ROWS * 128) + row * 128 + (((((col8 & 31) >> 3)) ^ (row & 3)) << 5);
    const float4 lo = *reinterpret_cast<const float4 *>(base), hi = *reinterpret_cast<const float4 *>(base + 16);
    f[0] = lo.x; f[1] = lo.y; f[2] = lo.z; f[3] = lo.w; f[4] = hi.x; f[5] = hi.y; f[6] = hi.z; f[7] = hi.w;
}

// ---- cumulative gates --------------------------------------------------------------------
// sLam holds NCH chunks of T rows x 64 channels (pitch kLamPitch) of gates; `scale` (log2(e) when
// the table holds raw gates) is applied while reading, so the sums are in log2 units.
// Turns every chunk's rows into inclusive prefix sums down the rows, in place; sLast[ch*64 + c]
// receives the last row (the chunk total).  NT threads; sTot has NT floats.
// Ends with a barrier.
// GROUP: the NT threads are only part of the CTA and synchronise with sync_group.
template <int NT, int NCH, bool GROUP = false>
__device__ __forceinline__ void gate_prefix(float *sLam, float *sLast, float *sTot, float scale = 1.f)
{
    constexpr int NSEG = NT / 64;                 // row segments over all NCH*T rows
    constexpr int R = NCH * T / NSEG;             // rows per segment
    constexpr int SEG_PER_CH = NSEG / NCH;
    static_assert(NSEG % NCH == 0 && R >= 1, "segments must not straddle chunks");
    const int c = threadIdx.x & 63, seg = threadIdx.x >> 6;
    float a[R];
#pragma unroll
    for (int j = 0; j < R; ++j) a[j] = sLam[(R * seg + j) * kLamPitch + c] * scale;
#pragma unroll
    for (int j = 1; j < R; ++j) a[j] += a[j - 1];
    sTot[seg * 64 + c] = a[R - 1];
    if (GROUP) sync_group(NT); else __syncthreads();
    const int first = (seg / SEG_PER_CH) * SEG_PER_CH;
    float add = 0.f;
#pragma unroll
    for (int s = 0; s < SEG_PER_CH - 1; ++s)
        if (first + s < seg) add += sTot[(first + s) * 64 + c];
#pragma unroll
    for (int j = 0; j < R; ++j) sLam[(R * seg + j) * kLamPitch + c] = a[j] + add;
    if (seg - first == SEG_PER_CH - 1) sLast[(seg / SEG_PER_CH) * 64 + c] = a[R - 1] + add;
    if (GROUP) sync_group(NT); else __syncthreads();
}

__device__ __forceinline__ void read_lam8(const float *sLam, int row, int col8, float (&lam)[8], bool flip = false)
{
    const int fl = flip ? 4 : 0;
    const float4 a = *reinterpret_cast<const float4 *>(sLam + row * kLamPitch + col8 + fl);
    const float4 b = *reinterpret_cast<const float4 *>(sLam + row * kLamPitch + col8 + 4 - fl);
    lam[0] = a.x; lam[1] = a.y; lam[2] = a.z; lam[3] = a.w; lam[4] = b.x; lam[5] = b.y; lam[6] = b.z; lam[7] = b.w;
}

// ---- MMA issue -----------------------------------------------------------------------------
// Descriptor of the first K-step of an operand tile; later K-steps add a constant.
//   K-format tile read K-major : 8 columns per step = 32 bytes inside the 128-byte row, a new
//                                column block (ROWS*128 bytes) every 4 steps.
//   M-format tile read MN-major: 8 rows per step = 1024 bytes.
template <int ROWS>
__device__ __forceinline__ uint64_t kdesc(const void *tile)
{
    return make_desc(smem_u32(tile), 16, 1024, 2);
}
template <int ROWS>
__device__ __forceinline__ uint64_t mdesc(const void *tile)
{
    return make_desc(smem_u32(tile), ROWS * 128, 512, 1);
}
template <int ROWS>
__device__ __forceinline__ uint64_t kstep(int kk)       // descriptor increment (16-byte units) of K-step kk
{
    return (uint64_t)((kk & 3) * 2 + (kk >> 2) * (ROWS * 8));
}
__device__ __forceinline__ uint64_t mstep(int kk) { return (uint64_t)(kk * 64); }

// D[tmem] (+)= A * B over KSTEPS steps of 8.  A_MN / B_MN: operand is an M-format tile read
// MN-major (contraction down its rows); otherwise a K-format tile read K-major.
template <int M, int N, bool A_MN, bool B_MN, int AROWS, int BROWS, int KSTEPS = 8>
__device__ __forceinline__ void issue(uint32_t d_tmem, uint64_t a0, uint64_t b0, bool accumulate)
{
    constexpr uint32_t idesc = idesc_tf32(M, N, A_MN, B_MN);
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
        const uint64_t da = a0 + (A_MN ? mstep(kk) : kstep<AROWS>(kk));
        const uint64_t db = b0 + (B_MN ? mstep(kk) : kstep<BROWS>(kk));
        mma_tf32(d_tmem, da, db, idesc, accumulate || kk > 0);
    }
}

__device__ __forceinline__ char *align1024(char *p)
{
    return reinterpret_cast<char *>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

struct Control {
    uint64_t bar[4];
    uint32_t tmem_base;
    uint32_t pad;
};
// bar[i] expects one arrival per phase, except bar[multi] (if >= 0), which expects multi_count.
__device__ __forceinline__ void setup(Control *ctl, int nbar, uint32_t tmem_cols, int multi = -1, int multi_count = 1)
{
    if (threadIdx.x < 32) tmem_alloc(&ctl->tmem_base, tmem_cols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < nbar; ++i) mbar_init(&ctl->bar[i], i == multi ? multi_count : 1);
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}
__device__ __forceinline__ void teardown(Control *ctl, uint32_t tmem_cols)
{
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(ctl->tmem_base, tmem_cols);
}

// 16 fp32 -> 16 bf16 (RNE) or 16 fp32, stored contiguously.
__device__ __forceinline__ void store16(float *p, const float (&v)[16])
{
#pragma unroll
    for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4 *>(p + 4 * j) = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}
__device__ __forceinline__ void store16(bf16 *p, const float (&v)[16])
{
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        uint4 u;
        __nv_bfloat162 t;
        t = __floats2bfloat162_rn(v[8 * j], v[8 * j + 1]); u.x = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]); u.y = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]); u.z = *reinterpret_cast<uint32_t *>(&t);
        t = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]); u.w = *reinterpret_cast<uint32_t *>(&t);
        *reinterpret_cast<uint4 *>(p + 8 * j) = u;
    }
}

// W accumulator values of row r, columns c0.. into a 64 x 64 state held in the swizzled tile order
// that the consuming kernels bulk-copy into shared memory (two column blocks of 64 rows x 128
// bytes, 16-byte pieces of a row XOR-ed with row & 7).
template <int W>
__device__ __forceinline__ void store_swizzled(float *state, int r, int c0, const float (&acc)[W])
{
    char *dst = reinterpret_cast<char *>(state);
#pragma unroll
    for (int j = 0; j < W / 4; ++j) {
        const int c = c0 + 4 * j;
        *reinterpret_cast<float4 *>(dst + (c >> 5) * (T * 128) + r * 128 + ((((c & 31) >> 2) ^ (r & 7)) << 4)) =
            make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
    }
}

}  // namespace tc
}  // namespace dig
