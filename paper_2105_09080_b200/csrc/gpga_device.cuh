// Device primitives for libgpga: Philox4x32-10, Box-Muller, streaming vector
// loads/stores and block reductions.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gpga {

// Round keys of Philox4x32-10 for one 64-bit seed: key word + r * Weyl constant,
// precomputed on the host so the kernels read them as launch constants.
struct PhiloxKeys {
    uint32_t k0[10];
    uint32_t k1[10];
};

__host__ __device__ inline PhiloxKeys make_philox_keys(uint32_t key0, uint32_t key1)
{
    PhiloxKeys ks;
    for (int r = 0; r < 10; ++r) {
        ks.k0[r] = key0 + (uint32_t)r * 0x9E3779B9u;
        ks.k1[r] = key1 + (uint32_t)r * 0xBB67AE85u;
    }
    return ks;
}

// Philox4x32-10 as published (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of
//   (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)),
// the key advancing by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& ks)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)c0 * 0xD2511F53ull;   // one 32x32->64 multiply each
        const uint64_t p1 = (uint64_t)c2 * 0xCD9E8D57ull;
        const uint32_t lo0 = (uint32_t)p0, hi0 = (uint32_t)(p0 >> 32);
        const uint32_t lo1 = (uint32_t)p1, hi1 = (uint32_t)(p1 >> 32);
        c0 = hi1 ^ c1 ^ ks.k0[r];
        c1 = lo1;
        c2 = hi0 ^ c3 ^ ks.k1[r];
        c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

__device__ __forceinline__ float fast_lg2(float x)
{
    float r;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float fast_sqrt(float x)
{
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float fast_sin(float x)
{
    float r;
    asm("sin.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float fast_cos(float x)
{
    float r;
    asm("cos.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// Box-Muller on one word pair.  u1 = ((a>>8)+1)/2^24 in (0,1], u2 = (b>>8)/2^24 in [0,1);
// returns (r cos 2 pi u2, r sin 2 pi u2), r = sqrt(-2 ln u1).
//  - Both uniforms are exact in fp32.
//  - Radius: the hardware log2 has an absolute error floor, which is a large
//    relative error where ln u1 -> 0; for 1 - u1 < 2^-10 the series
//    -ln(1 - t) = t + t^2/2 + t^3/3 (t exact) is used instead.
//  - Angle: evaluated at 2 pi (u2 - 1/2) in [-pi, pi), where the hardware sine and
//    cosine are most accurate, then negated (cos(x + pi) = -cos x).
// -2 ln u1 for u1 within 2^-10 of 1, from t = 1 - u1 = (2^24 - 1 - m) / 2^24 (exact): the series
// -ln(1 - t) = t + t^2/2 + t^3/3.  Needed by one sample in a thousand, so it is kept out of line:
// the common path does not carry its instructions.
static __device__ __noinline__ float neg2ln_near_one(uint32_t m)
{
    const float t = (float)(0xFFFFFFu - m) * 0x1p-24f;
    return t * (2.0f + t * (1.0f + t * 0.6666667f));
}

__device__ __forceinline__ float2 box_muller(uint32_t a, uint32_t b)
{
    const uint32_t m = a >> 8;
    // (the exact scaling to (0,1] first: the hardware log2 is most accurate near 1)
    const float u1 = (float)(m + 1u) * 0x1p-24f;
    float neg2ln = -1.3862943611198906f * fast_lg2(u1);
    if (m >= 0xFFFFFFu - 0x3FFFu) neg2ln = neg2ln_near_one(m);
    const float r = fast_sqrt(neg2ln);
    const float ang = (float)((int)(b >> 8) - (1 << 23)) * 3.7450704e-07f;   // 2 pi / 2^24
    return make_float2(-r * fast_cos(ang), -r * fast_sin(ang));
}

// Four standard normals for columns 4q..4q+3 of node i at iteration k.
__device__ __forceinline__ float4 normal4(uint32_t q, uint32_t i, uint32_t k, uint32_t stream,
                                          const PhiloxKeys& ks)
{
    const uint4 w = philox4x32_10(q, i, k, stream, ks);
    const float2 za = box_muller(w.x, w.y);
    const float2 zb = box_muller(w.z, w.w);
    return make_float4(za.x, za.y, zb.x, zb.y);
}

// Row index of the t-th mini-batch draw of node i at iteration k (drawn with replacement):
// word t & 3 of the generator call with counter (t >> 2, i, k, stream 4), reduced mod m.
__device__ __forceinline__ uint32_t batch_row(uint32_t t, uint32_t i, uint32_t k, uint32_t m,
                                              const PhiloxKeys& ks)
{
    const uint4 w = philox4x32_10(t >> 2, i, k, 4u, ks);
    const uint32_t sel = t & 3u;
    const uint32_t word = sel == 0 ? w.x : sel == 1 ? w.y : sel == 2 ? w.z : w.w;
    return word % m;
}

__device__ __forceinline__ float warp_sum_f(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// ---- packed pairs of fp32 (two IEEE fused multiply-adds per instruction on sm_100) ----------
// Each half is rounded exactly as a scalar fmaf of the same operands.
typedef unsigned long long f32x2_t;
__device__ __forceinline__ f32x2_t pack2(float lo, float hi)
{
    f32x2_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ float2 unpack2(f32x2_t v)
{
    float2 r;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(r.x), "=f"(r.y) : "l"(v));
    return r;
}
__device__ __forceinline__ f32x2_t fma2(f32x2_t a, f32x2_t b, f32x2_t c)
{
    f32x2_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

__device__ __forceinline__ f32x2_t add2(f32x2_t a, f32x2_t b)
{
    f32x2_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2_t sub2(f32x2_t a, f32x2_t b)
{
    f32x2_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2_t mul2(f32x2_t a, f32x2_t b)
{
    f32x2_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// Element-wise arithmetic on a group of four columns, two packed instructions each; every
// component is rounded as the scalar operation of the same name would round it.
__device__ __forceinline__ float4 join4(f32x2_t lo, f32x2_t hi)
{
    const float2 a = unpack2(lo), b = unpack2(hi);
    return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ float4 add4(float4 a, float4 b)
{
    return join4(add2(pack2(a.x, a.y), pack2(b.x, b.y)), add2(pack2(a.z, a.w), pack2(b.z, b.w)));
}
__device__ __forceinline__ float4 sub4(float4 a, float4 b)
{
    return join4(sub2(pack2(a.x, a.y), pack2(b.x, b.y)), sub2(pack2(a.z, a.w), pack2(b.z, b.w)));
}
__device__ __forceinline__ float4 scale4(float4 a, float s)
{
    const f32x2_t s2 = pack2(s, s);
    return join4(mul2(pack2(a.x, a.y), s2), mul2(pack2(a.z, a.w), s2));
}
// s * a + b
__device__ __forceinline__ float4 fma4(float s, float4 a, float4 b)
{
    const f32x2_t s2 = pack2(s, s);
    return join4(fma2(s2, pack2(a.x, a.y), pack2(b.x, b.y)), fma2(s2, pack2(a.z, a.w), pack2(b.z, b.w)));
}

// ---- streaming (read-once / write-once) 128-bit accesses -------------------
__device__ __forceinline__ float4 ld_stream4(const float* p)
{
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream4(float* p, float4 v)
{
    __stcs(reinterpret_cast<float4*>(p), v);
}

// Row access for one group of four columns starting at local column j0.
// VEC: d % 4 == 0 and 16-byte aligned bases -> one 128-bit access.  Otherwise
// four guarded scalar accesses (the last group of a row may be partial and rows
// are not 16-byte aligned).
template <bool VEC>
__device__ __forceinline__ float4 load4(const float* row, long long j0, long long d)
{
    if (VEC) return ld_stream4(row + j0);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j0 + 0 < d) v.x = __ldcs(row + j0 + 0);
    if (j0 + 1 < d) v.y = __ldcs(row + j0 + 1);
    if (j0 + 2 < d) v.z = __ldcs(row + j0 + 2);
    if (j0 + 3 < d) v.w = __ldcs(row + j0 + 3);
    return v;
}
template <bool VEC>
__device__ __forceinline__ void store4(float* row, long long j0, long long d, float4 v)
{
    if (VEC) {
        st_stream4(row + j0, v);
        return;
    }
    if (j0 + 0 < d) __stcs(row + j0 + 0, v.x);
    if (j0 + 1 < d) __stcs(row + j0 + 1, v.y);
    if (j0 + 2 < d) __stcs(row + j0 + 2, v.z);
    if (j0 + 3 < d) __stcs(row + j0 + 3, v.w);
}

// ---- block reduction of a double (warp shuffles, then one warp) ------------
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
// All threads of the block must call; result valid in thread 0.  blockDim.x <= 1024.
__device__ __forceinline__ double block_sum(double v)
{
    __shared__ double warp_part[32];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = warp_sum(v);
    if (lane == 0) warp_part[wid] = v;
    __syncthreads();
    const int nw = (blockDim.x + 31) >> 5;
    v = (threadIdx.x < nw) ? warp_part[threadIdx.x] : 0.0;
    if (wid == 0) v = warp_sum(v);
    __syncthreads();
    return v;
}

}  // namespace gpga
