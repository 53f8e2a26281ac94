// Shared device helpers for the CSD verification kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace csd {

constexpr int kThreads = 256;              // threads per block
constexpr int kWarps = kThreads / 32;      // independent streaming workers per block
constexpr int kUnroll = 8;                 // 16-byte vectors in flight per lane
constexpr float kLog2e = 1.4426950408889634f;
// Stand-in exponent reference of an accumulator that has seen no finite value yet:
// finite (so differences never produce inf - inf) and far below any real reference.
constexpr float kNoRef = -3.0e38f;
constexpr unsigned kFull = 0xffffffffu;

// One partial reduction of a contiguous run of logits.
//   m   : maximum of the run (-inf if the run holds no finite value)
//   idx : lowest element index (within the row) attaining m
//   c   : integer-valued reference exponent, c = rint(m * log2 e)
//   s   : sum over the run of 2^(x * log2 e - c)
// Keeping the reference an integer makes every rescale between partials an exact
// power-of-two multiplication, so sums combine without extra rounding and the
// only per-element rounding is the one in fma(x, log2 e, -c).
struct __align__(16) Partial {
    float m;
    int idx;
    float c;
    float s;
};

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Packed pairs of floats in one 64-bit register: sm_100 executes fma/add on both halves with
// one instruction (fma.rn.f32x2 / add.rn.f32x2), which halves the issue slots of the
// per-element multiply-add and accumulate.  Each half is rounded exactly like the scalar op.
__device__ __forceinline__ unsigned long long pack2(float lo, float hi)
{
    unsigned long long r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

__device__ __forceinline__ void unpack2(unsigned long long v, float &lo, float &hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c)
{
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b)
{
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

__device__ __forceinline__ unsigned long long mul2(unsigned long long a, unsigned long long b)
{
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// acc += (2^(x0*log2e - c), 2^(x1*log2e - c)) for a pair of logits
__device__ __forceinline__ void accum_pair(float x0, float x1, unsigned long long l2e2, unsigned long long negc2,
                                           unsigned long long &acc)
{
    float t0, t1;
    unpack2(fma2(pack2(x0, x1), l2e2, negc2), t0, t1);
    acc = add2(acc, pack2(ex2_approx(t0), ex2_approx(t1)));
}

// 2^k for an integer-valued k <= 0 (any value <= -127, -inf or NaN gives 0): exact.
__device__ __forceinline__ float pow2_nonpos(float k)
{
    k = fmaxf(k, -127.0f);          // NaN -> -127
    k = fminf(k, 0.0f);
    return __int_as_float((static_cast<int>(k) + 127) << 23);
}

__device__ __forceinline__ Partial partial_identity()
{
    Partial p;
    p.m = -INFINITY;
    p.idx = 0x7fffffff;
    p.c = kNoRef;
    p.s = 0.0f;
    return p;
}

// Combine two partials; `a` covers lower element indices than `b`.
__device__ __forceinline__ Partial combine(const Partial &a, const Partial &b)
{
    Partial r;
    const bool take_b = (b.m > a.m) || (b.m == a.m && b.idx < a.idx);
    r.m = take_b ? b.m : a.m;
    r.idx = take_b ? b.idx : a.idx;
    r.c = fmaxf(a.c, b.c);
    r.s = a.s * pow2_nonpos(a.c - r.c) + b.s * pow2_nonpos(b.c - r.c);
    return r;
}

__device__ __forceinline__ Partial shfl_up_partial(const Partial &p, int delta)
{
    Partial r;
    r.m = __shfl_up_sync(kFull, p.m, delta);
    r.idx = __shfl_up_sync(kFull, p.idx, delta);
    r.c = __shfl_up_sync(kFull, p.c, delta);
    r.s = __shfl_up_sync(kFull, p.s, delta);
    return r;
}

__device__ __forceinline__ Partial shfl_partial(const Partial &p, int src)
{
    Partial r;
    r.m = __shfl_sync(kFull, p.m, src);
    r.idx = __shfl_sync(kFull, p.idx, src);
    r.c = __shfl_sync(kFull, p.c, src);
    r.s = __shfl_sync(kFull, p.s, src);
    return r;
}

// 16-byte streaming load: read-only path, no L1 allocation (every logit is read once).
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// L2-coherent loads/stores for data exchanged between blocks of one launch.
__device__ __forceinline__ Partial ld_partial_cg(const Partial *p)
{
    const float4 v = __ldcg(reinterpret_cast<const float4 *>(p));
    Partial r;
    r.m = v.x;
    r.idx = __float_as_int(v.y);
    r.c = v.z;
    r.s = v.w;
    return r;
}

__device__ __forceinline__ void st_partial_cg(Partial *p, const Partial &v)
{
    __stcg(reinterpret_cast<float4 *>(p), make_float4(v.m, __int_as_float(v.idx), v.c, v.s));
}

}  // namespace csd
