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
// never contracted into an FMA).  With a layer table (LAYERS), an element of a
// layer with multipliers (lm, dm) uses  t = lm * (acc + (dm*d)*theta)  instead.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace softsync {

constexpr int kMaxFuseT = 16;
constexpr int kMaxReplicas = 8;

// Per-layer learning-rate / decay multipliers: layer q ends before element end[q].
template <int MAXSEG>
struct LayerTable {
    int count;
    long long end[MAXSEG];
    float lm[MAXSEG];
    float dm[MAXSEG];
};

// Everything one launch needs, passed by value in kernel-parameter space: the
// per-gradient scales s (Eq. 3 folded with the 1/c of Eq. 2), the per-group
// decay coefficients d and the borrowed gradient pointers, group-major.
template <int MAXE, int MAXSEG>
struct LaunchParams {
    float *w;
    float *v;
    long long n;          // elements
    float2 momentum;      // every coefficient is held twice (.x == .y), so that a packed multiply can take the
                          // pair as ONE 64-bit operand straight from parameter space
    int T;                // groups in this pass
    int c;                // gradients per group
    int overlap;          // 1: launched as a programmatic dependent; gradients may be fetched early
    int reverse;          // 1: blocks walk the vector from its end (alternates from launch to launch)
    unsigned short *mirror;   // optional bf16 copy of theta, rewritten by every pass (nullptr: none)
    int nrep;                 // further fp32 copies of this range of theta, written by the same pass: the weight
    float *rep[kMaxReplicas]; // broadcast of a sharded server (a destination may be another GPU's memory)
    float2 d[kMaxFuseT];
    float2 s[MAXE];
    const void *g[MAXE];
    LayerTable<MAXSEG> layers;    // used by the LAYERS instantiations only (MAXSEG = 1 otherwise)
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

// theta into its replicas.  Plain stores: a replica may live in a peer GPU's memory, where they travel as
// ordinary remote writes over NVLink (no load ever touches a replica).
template <int VEC, typename Params>
__device__ __forceinline__ void store_replicas(const Params &p, long long first, const float (&x)[VEC])
{
    for (int r = 0; r < p.nrep; ++r) {
        float *dst = p.rep[r] + first;
        if constexpr (VEC == 1) {
            *dst = x[0];
        } else {
            static_assert(VEC == 4, "fragments hold one or four elements");
            *reinterpret_cast<float4 *>(dst) = make_float4(x[0], x[1], x[2], x[3]);
        }
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
    float lm, dm;                     // the fragment's layer multipliers (LAYERS instantiations)
    int l, t;                         // position inside the current group, group index
};

// Index of the layer that holds element k: the first layer whose end lies beyond k.
template <int MAXSEG>
__device__ __forceinline__ int find_layer(const LayerTable<MAXSEG> &tab, long long k)
{
    int lo = 0, hi = tab.count - 1;                       // the last layer ends at n > k
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (tab.end[mid] > k) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// Packed fp32 pairs (sm_100 f32x2).  One packed multiply or subtract rounds each half exactly like its
// scalar form and costs one issue slot for two elements.  Only multiplies whose results feed SCALAR adds, and
// subtracts whose operands are not products, are packed: a packed multiply feeding a packed add is contracted
// into a fused multiply-add by ptxas 12.9 (single rounding), which the arithmetic contract forbids.
__device__ __forceinline__ void mul_pair(float &x0, float &x1, float a, float b0, float b1)
{
    unsigned long long A, B, R;
    asm("mov.b64 %0, {%1,%1};" : "=l"(A) : "f"(a));
    asm("mov.b64 %0, {%1,%2};" : "=l"(B) : "f"(b0), "f"(b1));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(R) : "l"(A), "l"(B));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(x0), "=f"(x1) : "l"(R));
}
__device__ __forceinline__ void sub_pair(float &x0, float &x1, float a0, float a1, float b0, float b1)
{
    unsigned long long A, B, R;
    asm("mov.b64 %0, {%1,%2};" : "=l"(A) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1,%2};" : "=l"(B) : "f"(b0), "f"(b1));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(R) : "l"(A), "l"(B));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(x0), "=f"(x1) : "l"(R));
}
// the same with the multiplier already a pair (a.x == a.y): a launch parameter
__device__ __forceinline__ void mul_pair(float &x0, float &x1, const float2 &a, float b0, float b1)
{
    unsigned long long A = *reinterpret_cast<const unsigned long long *>(&a), B, R;
    asm("mov.b64 %0, {%1,%2};" : "=l"(B) : "f"(b0), "f"(b1));
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(R) : "l"(A), "l"(B));
    asm("mov.b64 {%0,%1}, %2;" : "=f"(x0), "=f"(x1) : "l"(R));
}
// x[j] = a * y[j], every product rounded once
template <int VEC>
__device__ __forceinline__ void scale(float (&x)[VEC], const float2 &a, const float (&y)[VEC])
{
    if constexpr (VEC == 4) {
        mul_pair(x[0], x[1], a, y[0], y[1]);
        mul_pair(x[2], x[3], a, y[2], y[3]);
    } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) x[j] = __fmul_rn(a.x, y[j]);
    }
}
template <int VEC>
__device__ __forceinline__ void scale(float (&x)[VEC], float a, const float (&y)[VEC])
{
    if constexpr (VEC == 4) {
        mul_pair(x[0], x[1], a, y[0], y[1]);
        mul_pair(x[2], x[3], a, y[2], y[3]);
    } else {
#pragma unroll
        for (int j = 0; j < VEC; ++j) x[j] = __fmul_rn(a, y[j]);
    }
}

// Adds gradient entry e (already in registers) to the fragment; when it is the
// last of its group, performs that group's weight update.  Branches are uniform
// across the grid (they depend on e and c only).  CT = 1: the launch has c = 1, known at
// compile time: every entry is a group of its own, entry e is group e, and the position
// counters and their branches disappear (they are a quarter of the instructions of a fused
// bf16 pass otherwise).  CT = 0: c is read from the launch parameters.
template <typename GT, int VEC, bool LAYERS, int CT = 0, typename Params>
__device__ __forceinline__ void consume(const Params &p, Fragment<VEC> &f, const Raw<GT, VEC> &r, int e)
{
    float g[VEC], prod[VEC];
    widen(r, g);
    scale<VEC>(prod, p.s[e], g);
    bool complete = true;
    int t = e;                                           // CT = 1: entry e is group e
    if constexpr (CT == 1) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) f.acc[j] = prod[j];
    } else {
        if (f.l == 0) {
#pragma unroll
            for (int j = 0; j < VEC; ++j) f.acc[j] = prod[j];
        } else {
#pragma unroll
            for (int j = 0; j < VEC; ++j) f.acc[j] = __fadd_rn(f.acc[j], prod[j]);
        }
        complete = ++f.l == p.c;
        if (complete) { t = f.t++; f.l = 0; }
    }
    if (complete) {                                      // group complete: one weight update
        float dw[VEC], mv[VEC], tt[VEC];
        if constexpr (LAYERS) scale<VEC>(dw, __fmul_rn(f.dm, p.d[t].x), f.w);
        else scale<VEC>(dw, p.d[t], f.w);
        scale<VEC>(mv, p.momentum, f.v);
#pragma unroll
        for (int j = 0; j < VEC; ++j) tt[j] = __fadd_rn(f.acc[j], dw[j]);
        if constexpr (LAYERS) scale<VEC>(tt, f.lm, tt);
#pragma unroll
        for (int j = 0; j < VEC; ++j) f.v[j] = __fadd_rn(mv[j], tt[j]);
        if constexpr (VEC == 4) {
            sub_pair(f.w[0], f.w[1], f.w[0], f.w[1], f.v[0], f.v[1]);
            sub_pair(f.w[2], f.w[3], f.w[2], f.w[3], f.v[2], f.v[3]);
        } else {
#pragma unroll
            for (int j = 0; j < VEC; ++j) f.w[j] = __fsub_rn(f.w[j], f.v[j]);
        }
    }
}

// VEC elements starting at element `first` (fragment index i).  The first EC
// gradient loads and the theta/v loads are issued back to back before anything
// is consumed, so every thread has (EC + 2) independent 16-byte requests in
// flight.  MORE = false: the launch has exactly EC entries and the code is
// straight-line (no spare registers held for a loop that never runs).
// MORE = true: entries beyond EC follow in chunks of K loads, the last few one by one.
template <typename GT, int VEC, int EC, bool MORE, int K, bool LAYERS, int CT = 0, typename Params>
__device__ __forceinline__ void update_fragment(const Params &p, long long i, long long first, float lm, float dm)
{
    Fragment<VEC> f;
    Raw<GT, VEC> head[EC > 0 ? EC : 1];
#pragma unroll
    for (int e = 0; e < EC; ++e) load_raw(head[e], p.g[e], i);
    if (p.overlap) griddep_wait();                       // theta and v are the previous update's output
    load_state<VEC>(p.w + first, f.w);
    load_state<VEC>(p.v + first, f.v);
    f.l = 0; f.t = 0; f.lm = lm; f.dm = dm;
#pragma unroll
    for (int e = 0; e < EC; ++e) consume<GT, VEC, LAYERS, CT>(p, f, head[e], e);
    if constexpr (MORE) {
        static_assert(CT == 0, "the compile-time group size is for straight-line launches only");
        const int E = p.T * p.c;
        int e0 = EC;
        for (; e0 + K <= E; e0 += K) {                   // full chunks: K independent loads, no predicates
            Raw<GT, VEC> raw[K];
#pragma unroll
            for (int k = 0; k < K; ++k) load_raw(raw[k], p.g[e0 + k], i);
#pragma unroll
            for (int k = 0; k < K; ++k) consume<GT, VEC, LAYERS>(p, f, raw[k], e0 + k);
        }
        for (; e0 < E; ++e0) {                           // fewer than K left
            Raw<GT, VEC> r;
            load_raw(r, p.g[e0], i);
            consume<GT, VEC, LAYERS>(p, f, r, e0);
        }
    }
    store_state<VEC>(p.w + first, f.w);
    store_state<VEC>(p.v + first, f.v);
    if (p.mirror) store_mirror<VEC>(p.mirror + first, f.w);
    if (p.nrep) store_replicas<VEC>(p, first, f.w);
}

// One element, any number of entries, with the layer looked up for that element.
template <typename GT, int K, bool LAYERS, typename Params>
__device__ __forceinline__ void update_element(const Params &p, long long k)
{
    float lm = 1.f, dm = 1.f;
    if constexpr (LAYERS) {
        const int q = find_layer(p.layers, k);
        lm = p.layers.lm[q]; dm = p.layers.dm[q];
    }
    update_fragment<GT, 1, 0, true, K, LAYERS>(p, k, k, lm, dm);
}

// One fragment of VEC elements per thread: the grid covers the vector exactly once
// (blocks * threads >= n / VEC).  No grid-stride loop: a loop around the fragment
// makes the compiler keep a second iteration's registers alive and costs a third
// of the occupancy.  The host guarantees T*c == EC (MORE = false) or T*c > EC
// (MORE = true), and c = 1 when CT = 1 (used without a layer table only).  The (n mod VEC)
// trailing elements are done one by one by the first threads of the grid.  LAYERS: the fragment's multipliers are looked up once;
// a fragment that straddles a layer boundary is done element by element.
template <typename GT, int VEC, int EC, bool MORE, int K, bool LAYERS, int MAXE, int MAXSEG, int CT = 0>
__global__ void softsync_update_kernel(const __grid_constant__ LaunchParams<MAXE, MAXSEG> p)
{
    const long long nfrag = p.n / VEC;
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (p.overlap) griddep_launch_dependents();          // the next pass may start filling free SM slots
    if (tid < nfrag) {
        // Successive launches walk the vector in opposite directions: the part of theta and v that the
        // previous launch touched last is still in the L2 and is the first thing this launch needs.
        const long long i = p.reverse ? nfrag - 1 - tid : tid;
        const long long first = i * VEC;
        if constexpr (LAYERS && VEC > 1) {
            const int q = find_layer(p.layers, first);
            if (p.layers.end[q] >= first + VEC) {
                update_fragment<GT, VEC, EC, MORE, K, true>(p, i, first, p.layers.lm[q], p.layers.dm[q]);
            } else {
                for (int j = 0; j < VEC; ++j) update_element<GT, K, true>(p, first + j);
            }
        } else if constexpr (LAYERS) {
            update_element<GT, K, true>(p, first);
        } else {
            update_fragment<GT, VEC, EC, MORE, K, false, CT>(p, i, first, 1.f, 1.f);
        }
    }
    if constexpr (VEC > 1) {
        const long long done = nfrag * VEC;
        if (tid < p.n - done) update_element<GT, K, LAYERS>(p, done + tid);
    }
}

// =====================================================================================
// Bulk-copy staged variant (PS_KERNEL_BULK): persistent blocks, each walking the tiles
// b, b + grid, b + 2*grid, ...  One thread issues, per tile, one cp.async.bulk for theta,
// one for v and one per gradient into a ring of shared-memory stages, all completing on
// that stage's mbarrier; every thread then takes its fragments from shared memory, runs
// the same consume() chain and stores theta and v straight to global memory.  One block
// per cluster, no multicast, sources are this GPU's memory only.
//
// Every wait is bounded: a thread that polls a stage's barrier wait_limit times without
// success votes to abort; the block then waits (bounded again) for the copies it still
// has in flight, writes a status record and returns.  The host reports it as an error.
// =====================================================================================
constexpr int kBulkMaxStages = 8;

struct BulkStatus {               // 16 bytes in pinned, device-mapped host memory
    int code;                     // 0: fine; 1: a copy barrier did not complete in time
    int block;
    int stage;
    int tile;                     // the block's own tile counter k (its k-th tile)
};

struct BulkPlan {
    long long ntiles;             // full tiles; elements beyond ntiles * tile_elems take the element path
    int tile_elems;               // power of two, >= 256
    int stages;
    int wait_limit;
    int selftest;                 // 1: block 0 announces 16 bytes more than it copies for its first tile
    BulkStatus *status;
};

__device__ __forceinline__ unsigned smem_addr(const void *p) { return static_cast<unsigned>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count)
{ asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory"); }
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes)
{ asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory"); }
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    // the last operand bounds how long one poll may suspend the thread (nanoseconds)
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(1000u) : "memory");
    return ok != 0;
}
// Polls at most `limit` times; false if the phase did not complete.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, int limit)
{
    for (int tries = 0; tries < limit; ++tries)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// Global -> this block's shared memory; size and both addresses are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(unsigned dst, const void *src, unsigned bytes, unsigned bar)
{
    asm volatile("cp.async.bulk.shared::cta.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void load_raw_shared(Raw<GradFp32, 4> &r, const unsigned char *tile, int frag)
{ r.q = reinterpret_cast<const float4 *>(tile)[frag]; }
__device__ __forceinline__ void load_raw_shared(Raw<GradBf16, 4> &r, const unsigned char *tile, int frag)
{ r.q = reinterpret_cast<const uint2 *>(tile)[frag]; }
__device__ __forceinline__ void load_raw_shared(Raw<GradFp32, 1> &r, const unsigned char *tile, int el)
{ r.q = reinterpret_cast<const float *>(tile)[el]; }
__device__ __forceinline__ void load_raw_shared(Raw<GradBf16, 1> &r, const unsigned char *tile, int el)
{ r.q = reinterpret_cast<const unsigned short *>(tile)[el]; }

// VEC elements of a staged tile: local index `li` (fragment index for VEC = 4, element index for VEC = 1),
// global element `first`.
template <typename GT, int VEC, bool LAYERS, typename Params>
__device__ __forceinline__ void update_from_stage(const Params &p, const unsigned char *stage, int tile_elems, int E,
                                                  int li, long long first, float lm, float dm)
{
    constexpr int GB = sizeof(Raw<GT, 1>);               // bytes per gradient element
    Fragment<VEC> f;
    const float *ws = reinterpret_cast<const float *>(stage);
    const float *vs = ws + tile_elems;
    const unsigned char *gs = stage + static_cast<size_t>(tile_elems) * 8;
#pragma unroll
    for (int j = 0; j < VEC; ++j) { f.w[j] = ws[li * VEC + j]; f.v[j] = vs[li * VEC + j]; }
    f.l = 0; f.t = 0; f.lm = lm; f.dm = dm;
    if (p.c == 1) {                                      // every entry its own update: no position counters
#pragma unroll 4
        for (int e = 0; e < E; ++e) {
            Raw<GT, VEC> r;
            load_raw_shared(r, gs + static_cast<size_t>(e) * tile_elems * GB, li);
            consume<GT, VEC, LAYERS, 1>(p, f, r, e);
        }
    } else {
#pragma unroll 4
        for (int e = 0; e < E; ++e) {
            Raw<GT, VEC> r;
            load_raw_shared(r, gs + static_cast<size_t>(e) * tile_elems * GB, li);
            consume<GT, VEC, LAYERS>(p, f, r, e);
        }
    }
    store_state<VEC>(p.w + first, f.w);
    store_state<VEC>(p.v + first, f.v);
    if (p.mirror) store_mirror<VEC>(p.mirror + first, f.w);
    if (p.nrep) store_replicas<VEC>(p, first, f.w);
}

// BLOCK_RECORDS: plan.status is an array with one record per block of the grid (each block that gives up
// writes its own) instead of one record shared by the launch.
template <typename GT, bool LAYERS, int MAXE, int MAXSEG, bool BLOCK_RECORDS = false>
__global__ void softsync_update_bulk_kernel(const __grid_constant__ LaunchParams<MAXE, MAXSEG> p,
                                            const __grid_constant__ BulkPlan plan)
{
    constexpr int GB = sizeof(Raw<GT, 1>);
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) unsigned long long full[kBulkMaxStages];

    const int E = p.T * p.c;
    const int S = plan.stages;
    const int tile = plan.tile_elems;
    const unsigned state_bytes = static_cast<unsigned>(tile) * 4u;
    const unsigned grad_bytes = static_cast<unsigned>(tile) * GB;
    const size_t stage_bytes = static_cast<size_t>(tile) * (8 + static_cast<size_t>(E) * GB);
    const long long G = gridDim.x, b = blockIdx.x;
    const long long mine = b < plan.ntiles ? (plan.ntiles - b + G - 1) / G : 0;    // tiles of this block

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) mbar_init(smem_addr(&full[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (p.overlap) griddep_launch_dependents();

    // element offset of this block's k-th tile
    auto tile_start = [&](long long k) {
        const long long t = b + k * G;
        return (p.reverse ? plan.ntiles - 1 - t : t) * static_cast<long long>(tile);
    };
    // the two halves of one tile's copies: gradients (inputs that exist already) and theta, v
    auto issue_grads = [&](long long k) {
        const int s = static_cast<int>(k % S);
        const unsigned bar = smem_addr(&full[s]);
        const long long off = tile_start(k);
        unsigned announce = 2u * state_bytes + static_cast<unsigned>(E) * grad_bytes;
        if (plan.selftest && b == 0 && k == 0) announce += 16u;
        mbar_expect_tx(bar, announce);
        unsigned char *dst = stage_mem + s * stage_bytes + static_cast<size_t>(tile) * 8;
        for (int e = 0; e < E; ++e)
            bulk_load(smem_addr(dst + static_cast<size_t>(e) * grad_bytes),
                      static_cast<const unsigned char *>(p.g[e]) + off * GB, grad_bytes, bar);
    };
    auto issue_state = [&](long long k) {
        const int s = static_cast<int>(k % S);
        const unsigned bar = smem_addr(&full[s]);
        const long long off = tile_start(k);
        unsigned char *dst = stage_mem + s * stage_bytes;
        bulk_load(smem_addr(dst), p.w + off, state_bytes, bar);
        bulk_load(smem_addr(dst + state_bytes), p.v + off, state_bytes, bar);
    };

    const long long prologue = mine < S ? mine : S;
    if (threadIdx.x == 0)
        for (long long k = 0; k < prologue; ++k) issue_grads(k);
    if (p.overlap) griddep_wait();                       // theta and v are the previous update's output
    if (threadIdx.x == 0)
        for (long long k = 0; k < prologue; ++k) issue_state(k);

    // elements behind the last full tile, one by one, by the block with the fewest tiles
    if (b == G - 1) {
        const long long done = plan.ntiles * static_cast<long long>(tile);
        for (long long k = done + threadIdx.x; k < p.n; k += blockDim.x) update_element<GT, 8, LAYERS>(p, k);
    }

    long long k = 0;
    bool gave_up = false;
    for (; k < mine; ++k) {
        const int s = static_cast<int>(k % S);
        const unsigned parity = static_cast<unsigned>((k / S) & 1);
        const bool arrived = mbar_wait_bounded(smem_addr(&full[s]), parity, plan.wait_limit);
        if (arrived) {
            const unsigned char *stage = stage_mem + s * stage_bytes;
            const long long base = tile_start(k);
            for (int fi = threadIdx.x; fi < tile / 4; fi += blockDim.x) {
                const long long first = base + 4ll * fi;
                if constexpr (LAYERS) {
                    const int q = find_layer(p.layers, first);
                    if (p.layers.end[q] >= first + 4) {
                        update_from_stage<GT, 4, true>(p, stage, tile, E, fi, first, p.layers.lm[q], p.layers.dm[q]);
                    } else {
                        for (int j = 0; j < 4; ++j) {
                            const int qj = find_layer(p.layers, first + j);
                            update_from_stage<GT, 1, true>(p, stage, tile, E, 4 * fi + j, first + j,
                                                           p.layers.lm[qj], p.layers.dm[qj]);
                        }
                    }
                } else {
                    update_from_stage<GT, 4, false>(p, stage, tile, E, fi, first, 1.f, 1.f);
                }
            }
        }
        // one barrier per tile: every thread is done reading stage s (it may be refilled), and the vote
        gave_up = __syncthreads_or(arrived ? 0 : 1) != 0;
        if (gave_up) break;
        if (threadIdx.x == 0 && k + S < mine) { issue_grads(k + S); issue_state(k + S); }
    }

    if (gave_up && threadIdx.x == 0) {
        // copies still in flight target this block's shared memory: wait for them (bounded) before leaving
        const long long issued = (k + S < mine) ? k + S : mine;     // tiles k .. issued-1 were issued and not consumed
        for (long long j = k; j < issued; ++j)
            mbar_wait_bounded(smem_addr(&full[j % S]), static_cast<unsigned>((j / S) & 1), plan.wait_limit);
        volatile BulkStatus *st = BLOCK_RECORDS ? plan.status + b : plan.status;
        st->block = static_cast<int>(b);
        st->stage = static_cast<int>(k % S);
        st->tile = static_cast<int>(k);
        __threadfence_system();
        st->code = 1;
        __threadfence_system();
    }
}

}  // namespace softsync
