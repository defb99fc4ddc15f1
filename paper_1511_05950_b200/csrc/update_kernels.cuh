// Fused sumGradients + applyUpdate kernels of the n-softsync parameter server
// (arXiv 1511.05950, Section 2.1; Eq. 2 with the per-gradient rate of Eq. 3).
//
// One pass over the parameter vector: every thread owns one fragment of VEC
// consecutive elements, loads theta and v once, streams the T*c gradient values
// of those elements through registers, applies the T updates in order and
// stores theta and v once.  The path is HBM-bound (about 0.3 flop per byte), so the work is
// plain fp32 ALU code around wide coalesced loads; tensor cores have no part.
//
// Arithmetic contract (bit-exact, any launch shape): per element and per group
//     acc = s_1*g_1;  acc = acc + s_l*g_l  (l = 2..c);
//     t = acc + d*theta;  v = m*v + t;  theta = theta - v
// with every multiply and add rounded separately (__fmul_rn / __fadd_rn are
// never contracted into an FMA).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace softsync {

constexpr int kMaxFuseT = 16;

// Everything one launch needs, passed by value in kernel-parameter space: the
// per-gradient scales s (Eq. 3 folded with the 1/c of Eq. 2), the per-group
// decay coefficients d and the borrowed gradient pointers, group-major.
template <int MAXE>
struct LaunchParams {
    float *w;
    float *v;
    long long n;          // elements
    float momentum;
    int T;                // groups in this pass
    int c;                // gradients per group
    int overlap;          // 1: launched as a programmatic dependent; gradients may be fetched early
    int reverse;          // 1: blocks walk the vector from its end (alternates from launch to launch)
    unsigned short *mirror;   // optional bf16 copy of theta, rewritten by every pass (nullptr: none)
    float d[kMaxFuseT];
    float s[MAXE];
    const void *g[MAXE];
};

struct GradFp32 {};
struct GradBf16 {};

// ---- raw gradient fragments: 4 elements (16 bytes fp32, 8 bytes bf16) or one ----
template <typename GT, int VEC> struct Raw;
template <> struct Raw<GradFp32, 4> { float4 q; };
template <> struct Raw<GradBf16, 4> { uint2 q; };
template <> struct Raw<GradFp32, 1> { float q; };
template <> struct Raw<GradBf16, 1> { unsigned short q; };

__device__ __forceinline__ float4 ld_stream_f4(const float4 *p)
{
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint2 ld_stream_u2(const uint2 *p)
{
    uint2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}

__device__ __forceinline__ void load_raw(Raw<GradFp32, 4> &r, const void *base, long long i)
{ r.q = ld_stream_f4(reinterpret_cast<const float4 *>(base) + i); }
__device__ __forceinline__ void load_raw(Raw<GradBf16, 4> &r, const void *base, long long i)
{ r.q = ld_stream_u2(reinterpret_cast<const uint2 *>(base) + i); }
__device__ __forceinline__ void load_raw(Raw<GradFp32, 1> &r, const void *base, long long i)
{ r.q = __ldg(reinterpret_cast<const float *>(base) + i); }
__device__ __forceinline__ void load_raw(Raw<GradBf16, 1> &r, const void *base, long long i)
{ r.q = __ldg(reinterpret_cast<const unsigned short *>(base) + i); }

// bf16 is the upper half of an fp32: widening is a shift, exact.
__device__ __forceinline__ void widen(const Raw<GradFp32, 4> &r, float (&g)[4])
{ g[0] = r.q.x; g[1] = r.q.y; g[2] = r.q.z; g[3] = r.q.w; }
__device__ __forceinline__ void widen(const Raw<GradBf16, 4> &r, float (&g)[4])
{
    g[0] = __uint_as_float(r.q.x << 16); g[1] = __uint_as_float(r.q.x & 0xFFFF0000u);
    g[2] = __uint_as_float(r.q.y << 16); g[3] = __uint_as_float(r.q.y & 0xFFFF0000u);
}
__device__ __forceinline__ void widen(const Raw<GradFp32, 1> &r, float (&g)[1]) { g[0] = r.q; }
__device__ __forceinline__ void widen(const Raw<GradBf16, 1> &r, float (&g)[1])
{ g[0] = __uint_as_float(static_cast<unsigned>(r.q) << 16); }

// ---- theta / v fragments ---------------------------------------------------
template <int VEC>
__device__ __forceinline__ void load_state(const float *p, float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        x[0] = *p;
    } else {
#pragma unroll
        for (int j = 0; j < VEC / 4; ++j) {
            const float4 q = __ldcs(reinterpret_cast<const float4 *>(p) + j);
            x[4 * j] = q.x; x[4 * j + 1] = q.y; x[4 * j + 2] = q.z; x[4 * j + 3] = q.w;
        }
    }
}
template <int VEC>
__device__ __forceinline__ void store_state(float *p, const float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        *p = x[0];
    } else {
#pragma unroll
        for (int j = 0; j < VEC / 4; ++j)
            __stcs(reinterpret_cast<float4 *>(p) + j, make_float4(x[4 * j], x[4 * j + 1], x[4 * j + 2], x[4 * j + 3]));
    }
}

// Programmatic dependent launch (sm_90+): a kernel launched with the stream-serialisation
// attribute may start while the previous kernel on the stream is draining; it must not touch
// that kernel's output before griddep_wait() returns.  Both are no-ops in an ordinary launch.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---- bf16 mirror of theta: round to nearest even, stored as raw 16-bit patterns ----
__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi)
{
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);       // .x = lo (low half), .y = hi
    return *reinterpret_cast<const unsigned *>(&b);
}
template <int VEC>
__device__ __forceinline__ void store_mirror(unsigned short *p, const float (&x)[VEC])
{
    if constexpr (VEC == 1) {
        *p = __bfloat16_as_ushort(__float2bfloat16_rn(x[0]));
    } else {
        static_assert(VEC == 4, "fragments hold one or four elements");
        __stcs(reinterpret_cast<uint2 *>(p), make_uint2(pack_bf16x2(x[0], x[1]), pack_bf16x2(x[2], x[3])));
    }
}

// theta -> bf16 mirror on its own (after ps_init_weights or when a mirror is bound).
__global__ void mirror_kernel(const float *w, unsigned short *mirror, long long n)
{
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n; i += stride)
        mirror[i] = __bfloat16_as_ushort(__float2bfloat16_rn(w[i]));
}

// ---- running state of one fragment while its gradients stream through -------
template <int VEC>
struct Fragment {
    float w[VEC], v[VEC], acc[VEC];
    int l, t;                         // position inside the current group, group index
};

// Adds gradient entry e (already in registers) to the fragment; when it is the
// last of its group, performs that group's weight update.  Branches are uniform
// across the grid (they depend on e and c only).
template <typename GT, int VEC, int MAXE>
__device__ __forceinline__ void consume(const LaunchParams<MAXE> &p, Fragment<VEC> &f, const Raw<GT, VEC> &r, int e)
{
    float g[VEC];
    widen(r, g);
    const float s = p.s[e];
    if (f.l == 0) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) f.acc[j] = __fmul_rn(s, g[j]);
    } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) f.acc[j] = __fadd_rn(f.acc[j], __fmul_rn(s, g[j]));
    }
    if (++f.l == p.c) {                                  // group complete: one weight update
        const float d = p.d[f.t++];
        const float m = p.momentum;
        f.l = 0;
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            const float tt = __fadd_rn(f.acc[j], __fmul_rn(d, f.w[j]));
            f.v[j] = __fadd_rn(__fmul_rn(m, f.v[j]), tt);
            f.w[j] = __fsub_rn(f.w[j], f.v[j]);
        }
    }
}

// VEC elements starting at element `first` (fragment index i).  The first EC
// gradient loads and the theta/v loads are issued back to back before anything
// is consumed, so every thread has (EC + 2) independent 16-byte requests in
// flight.  MORE = false: the launch has exactly EC entries and the code is
// straight-line (no spare registers held for a loop that never runs).
// MORE = true: entries beyond EC follow in chunks of K loads, the last few one by one.
template <typename GT, int VEC, int EC, bool MORE, int K, int MAXE>
__device__ __forceinline__ void update_fragment(const LaunchParams<MAXE> &p, long long i, long long first)
{
    Fragment<VEC> f;
    Raw<GT, VEC> head[EC > 0 ? EC : 1];
#pragma unroll
    for (int e = 0; e < EC; ++e) load_raw(head[e], p.g[e], i);
    if (p.overlap) griddep_wait();                       // theta and v are the previous update's output
    load_state<VEC>(p.w + first, f.w);
    load_state<VEC>(p.v + first, f.v);
    f.l = 0; f.t = 0;
#pragma unroll
    for (int e = 0; e < EC; ++e) consume<GT, VEC, MAXE>(p, f, head[e], e);
    if constexpr (MORE) {
        const int E = p.T * p.c;
        int e0 = EC;
        for (; e0 + K <= E; e0 += K) {                   // full chunks: K independent loads, no predicates
            Raw<GT, VEC> raw[K];
#pragma unroll
            for (int k = 0; k < K; ++k) load_raw(raw[k], p.g[e0 + k], i);
#pragma unroll
            for (int k = 0; k < K; ++k) consume<GT, VEC, MAXE>(p, f, raw[k], e0 + k);
        }
        for (; e0 < E; ++e0) {                           // fewer than K left
            Raw<GT, VEC> r;
            load_raw(r, p.g[e0], i);
            consume<GT, VEC, MAXE>(p, f, r, e0);
        }
    }
    store_state<VEC>(p.w + first, f.w);
    store_state<VEC>(p.v + first, f.v);
    if (p.mirror) store_mirror<VEC>(p.mirror + first, f.w);
}

// One fragment of VEC elements per thread: the grid covers the vector exactly once
// (blocks * threads >= n / VEC).  No grid-stride loop: a loop around the fragment
// makes the compiler keep a second iteration's registers alive and costs a third
// of the occupancy.  The host guarantees T*c == EC (MORE = false) or T*c > EC
// (MORE = true).  The (n mod VEC) trailing elements are done one by one by the
// first threads of the grid.
template <typename GT, int VEC, int EC, bool MORE, int K, int MAXE>
__global__ void softsync_update_kernel(const __grid_constant__ LaunchParams<MAXE> p)
{
    const long long nfrag = p.n / VEC;
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (p.overlap) griddep_launch_dependents();          // the next pass may start filling free SM slots
    if (tid < nfrag) {
        // Successive launches walk the vector in opposite directions: the part of theta and v that the
        // previous launch touched last is still in the L2 and is the first thing this launch needs.
        const long long i = p.reverse ? nfrag - 1 - tid : tid;
        update_fragment<GT, VEC, EC, MORE, K, MAXE>(p, i, i * VEC);
    }
    if constexpr (VEC > 1) {
        const long long done = nfrag * VEC;
        if (tid < p.n - done)
            update_fragment<GT, 1, 0, true, K, MAXE>(p, done + tid, done + tid);
    }
}

}  // namespace softsync
