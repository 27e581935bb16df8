// kt_kernels.cuh -- device tables and sm_100a kernels of the hierarchical, load-weighted
// gradient synchronisation (paper Section III-A: intra-group reduce, fp32 transport,
// inter-group combine; Section III-C supplies the weights).
//
// Work decomposition.  The fp32 transport is cut into tiles of TILE elements that never
// cross a tensor boundary; one CTA handles one tile (the grid is the tile count, so the
// hardware scheduler balances ragged tensor lists and partial waves by itself).  A CTA
// finds its tensor in the per-tensor tile prefix (one thread per tensor), then streams the K rank
// buffers of that tile with 128-bit loads, all loads of a batch of ranks issued before the
// first multiply.  Interior tiles of 16-byte aligned tensors run without predicates; tiles
// that hold a tensor's tail, zero padding, or a misaligned tensor use the same code with
// per-vector predicates and element loads only where a vector would cross the end.
//
// Arithmetic order is fixed: first member of a group acc = a*x (one rounded multiply),
// later members acc = fma(a, x, acc); the same across groups with W_g.
#pragma once

#include <cuda_runtime.h>

#include "../../include/kaitian.h"

namespace {

#ifndef KT_NT
#define KT_NT 256
#endif
#ifndef KT_ITERS
#define KT_ITERS 2
#endif
#ifndef KT_KB
#define KT_KB 4                  /* ranks whose loads are issued together */
#endif
#ifndef KT_KB_DIRECT_BF16
#define KT_KB_DIRECT_BF16 2      /* the same for the direct path on bf16 gradients (keeps it at 4 CTAs per SM) */
#endif
constexpr int NT = KT_NT;        // threads per CTA
// transport elements per work unit (one CTA each): chosen by the gradient dtype so that every
// thread has KT_ITERS 16-byte loads per rank in flight
constexpr int TILE_F32 = NT * 4 * KT_ITERS;
constexpr int TILE_BF16 = NT * 8 * KT_ITERS;
constexpr int FLAG_ALIGNED = 1;  // all K sources of the tensor are 16-byte aligned

// ------------------------------------------------------------------ device tables
struct TInfo {            // one per tensor, transport order
    long long dst_off;    // element offset in the transport
    long long numel;      // gradient elements
    long long ext;        // numel + zero padding up to the next tensor (a multiple of 8)
    int flags;
    int pad_;
};

struct RankTab {          // ranks in group-major order (ascending rank inside a group)
    float coef[KT_MAX_RANKS];
    signed char gid[KT_MAX_RANKS];
    unsigned char first[KT_MAX_RANKS];   // first member of its group
    unsigned char last[KT_MAX_RANKS];    // last member of its group
    int K;
};

struct GroupTab {
    float W[KT_MAX_GROUPS];
    int G;
};

struct TilePlan {         // which tiles a launch covers and how to decode them
    const int *prefix;    // [T+1] tiles before tensor u
    const TInfo *info;    // [T]
    int T;
    int u_lo, u_hi;       // tensors [u_lo, u_hi) take part
    int tile_lo;          // first tile of the launch: prefix[u_lo], or later when a device's share starts mid-tensor
    int n_tiles;          // tiles of the launch (it may end before prefix[u_hi] for the same reason)
    int tile;             // elements per tile the prefix was built for
    int single;           // the launch covers (part of) exactly one tensor: its record travels in `one`
    TInfo one;            // ... and the fused reduce decodes its tiles by arithmetic, without any table
    int single_skip;      // ... starting this many tiles into the tensor (a device's share may begin mid-tensor)
};

struct K1Params {
    TilePlan tp;
    const void *const *ptrs;           // [K][T] device pointer table
    void *transport[KT_MAX_GROUPS];    // fp32, or bf16 when the context's transport is narrowed
    RankTab rt;
    int wide;                          // every transport base is 32-byte aligned
};

struct K2Params {
    TilePlan tp;
    const void *src[KT_MAX_GROUPS];    // partials (fp32 or bf16 transport), or one fp32 combined buffer
    GroupTab gt;
    void *const *out_ptrs;             // [R][T] device pointer table
    const unsigned char *out_aligned;  // [T] all R destinations 16-byte aligned
    int R;
    float scale;
    int wide;                          // every source base is 32-byte aligned
};

struct DirectParams {
    TilePlan tp;
    const void *const *ptrs;           // [K][T] device pointer table
    RankTab rt;
    GroupTab gt;
    void *const *out_ptrs;             // [R][T] device pointer table
    const unsigned char *out_aligned;  // [T] all R destinations 16-byte aligned
    int R;
    float scale;
};

struct BcastParams {
    TilePlan tp;
    void *const *ptrs;                     // [K][T] registered tensors, group-major rank order
    void *flat[KT_MAX_GROUPS];             // send: [g_root] is written; recv: [g != g_root] are read
    unsigned char k_lo[KT_MAX_GROUPS];     // members of group g: ranks [k_lo[g], k_hi[g]) of that order
    unsigned char k_hi[KT_MAX_GROUPS];
    int G, g_root, k_root;
};

struct PackParams {
    TilePlan tp;
    const void *const *ptrs;           // [K][T], group-major rank order
    void *flat[KT_MAX_RANKS];          // same rank order
    int K;
};

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ uint4 ld_stream(const void *p) {
    // read-once data: keep it out of L1
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint4 ld_plain(const void *p) {
    // for data the same launch also writes (in-place outputs): an ordinary, coherent load
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}

template <typename P>
__device__ __forceinline__ P *ldg_ptr(P *const *slot) {
    // pointer tables are read-only for the lifetime of a launch
    return reinterpret_cast<P *>(__ldg(reinterpret_cast<const unsigned long long *>(slot)));
}

__device__ __forceinline__ unsigned pack_bf16x2(float lo, float hi) {
    unsigned d;   // round-to-nearest-even narrowing of two floats; hi lands in the upper half
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// VEC consecutive floats to / from the transport.  Eight floats go as one 256-bit access when
// the buffers allow it (32-byte aligned bases), so that every access covers whole 32-byte
// sectors; otherwise as two 128-bit accesses.
template <int VEC>
__device__ __forceinline__ void store_vec(float *d, const float (&a)[VEC], bool wide) {
    if (VEC == 8 && wide) {
        asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(d), "f"(a[0]), "f"(a[1]),
                     "f"(a[2]), "f"(a[3]), "f"(a[4 % VEC]), "f"(a[5 % VEC]), "f"(a[6 % VEC]), "f"(a[7 % VEC])
                     : "memory");
    } else {
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q)
            reinterpret_cast<float4 *>(d)[q] = make_float4(a[4 * q], a[4 * q + 1], a[4 * q + 2], a[4 * q + 3]);
    }
}

template <int Q>
__device__ __forceinline__ void load_vec(const float *s, float4 (&v)[Q], bool wide) {
    if (Q == 2 && wide) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[0].z), "=f"(v[0].w), "=f"(v[Q - 1].x), "=f"(v[Q - 1].y),
                       "=f"(v[Q - 1].z), "=f"(v[Q - 1].w)
                     : "l"(s));
    } else {
#pragma unroll
        for (int q = 0; q < Q; ++q) v[q] = __ldcs(reinterpret_cast<const float4 *>(s) + q);
    }
}

// The same for a transport of type TT (float, or unsigned short = bf16): VEC partial sums are
// written as they are or narrowed to nearest-even; VEC transport elements are read and widened.
template <typename TT, int VEC>
__device__ __forceinline__ void store_transport(void *base, long long at, const float (&a)[VEC], bool wide) {
    if constexpr (sizeof(TT) == 4) {
        store_vec<VEC>(static_cast<float *>(base) + at, a, wide);
    } else {
        unsigned short *d = static_cast<unsigned short *>(base) + at;
        if constexpr (VEC == 8)
            *reinterpret_cast<uint4 *>(d) = make_uint4(pack_bf16x2(a[0], a[1]), pack_bf16x2(a[2], a[3]),
                                                       pack_bf16x2(a[4], a[5]), pack_bf16x2(a[6], a[7]));
        else
            *reinterpret_cast<uint2 *>(d) = make_uint2(pack_bf16x2(a[0], a[1]), pack_bf16x2(a[2], a[3]));
    }
}

template <typename TT, int VEC>
__device__ __forceinline__ void load_transport(const void *base, long long at, float (&x)[VEC], bool wide) {
    if constexpr (sizeof(TT) == 4) {
        float4 v[VEC / 4];
        load_vec<VEC / 4>(static_cast<const float *>(base) + at, v, wide);
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q) {
            x[4 * q] = v[q].x; x[4 * q + 1] = v[q].y; x[4 * q + 2] = v[q].z; x[4 * q + 3] = v[q].w;
        }
    } else {
        const unsigned short *s = static_cast<const unsigned short *>(base) + at;
        unsigned w[VEC / 2];
        if constexpr (VEC == 8) {
            const uint4 v = ld_stream(s);
            w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
        } else {
            asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(s));
        }
#pragma unroll
        for (int q = 0; q < VEC / 2; ++q) {
            x[2 * q] = __uint_as_float(w[q] << 16);
            x[2 * q + 1] = __uint_as_float(w[q] & 0xFFFF0000u);
        }
    }
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int VEC = 4;   // elements per 16-byte vector
    static constexpr int TILE = TILE_F32;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&x)[4]) {
        x[0] = __uint_as_float(v.x); x[1] = __uint_as_float(v.y);
        x[2] = __uint_as_float(v.z); x[3] = __uint_as_float(v.w);
    }
    // elements [e, e + 4) of s that lie below n, zero elsewhere
    __device__ static __forceinline__ uint4 gather(const float *s, long long e, long long n) {
        unsigned w[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) w[c] = (e + c < n) ? __float_as_uint(s[e + c]) : 0u;
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    __device__ static __forceinline__ uint4 narrow(const float (&y)[4]) {
        return make_uint4(__float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]),
                          __float_as_uint(y[3]));
    }
    __device__ static __forceinline__ float narrow_one(float y) { return y; }
};
template <> struct Elem<unsigned short> {
    static constexpr int VEC = 8;
    static constexpr int TILE = TILE_BF16;
    __device__ static __forceinline__ void unpack(const uint4 &v, float (&x)[8]) {
        // bf16 is the upper half of a binary32: widening is a shift
        x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xFFFF0000u);
        x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xFFFF0000u);
        x[4] = __uint_as_float(v.z << 16); x[5] = __uint_as_float(v.z & 0xFFFF0000u);
        x[6] = __uint_as_float(v.w << 16); x[7] = __uint_as_float(v.w & 0xFFFF0000u);
    }
    __device__ static __forceinline__ uint4 gather(const unsigned short *s, long long e, long long n) {
        unsigned w[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const unsigned lo = (e + 2 * c < n) ? s[e + 2 * c] : 0u;
            const unsigned hi = (e + 2 * c + 1 < n) ? s[e + 2 * c + 1] : 0u;
            w[c] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    __device__ static __forceinline__ uint4 narrow(const float (&y)[8]) {
        return make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]), pack_bf16x2(y[4], y[5]),
                          pack_bf16x2(y[6], y[7]));
    }
    __device__ static __forceinline__ unsigned short narrow_one(float y) {
        return static_cast<unsigned short>(pack_bf16x2(y, 0.f) & 0xFFFFu);
    }
};

// What a CTA works on: tensor u (transport order), its record, first element of the tile.
struct TileRef {
    int u;
    TInfo ti;
    long long e0;
};

// Tile -> tensor: the u with prefix[u] <= tile < prefix[u + 1] (prefix is non-decreasing, so
// empty tensors never match).  One memory round trip: thread i tests tensor u_lo + i (in
// strides of the CTA when there are more tensors than threads), the one that matches
// publishes it through shared memory.  (Prefetching the tables into L2 by the first CTAs of a
// launch was measured and taken out: it cost 1-4 % on the named workloads and 14 % on the
// combine of the ragged MobileNetV2 list.)  SINGLE_SHORTCUT: a launch that covers
// exactly one tensor (flat buffers, one-tensor buckets) carries that tensor's record in its
// parameters and decodes tiles by arithmetic, with no table access at all (used by the fused
// reduce, where it measured 1-8 % faster on flat buffers; the other kernels did not gain).
// `bid`: which tile of the launch this CTA takes (its block index unless the kernel says otherwise).
template <bool SINGLE_SHORTCUT = false>
__device__ __forceinline__ TileRef locate_tile(const TilePlan &tp, unsigned bid = blockIdx.x) {
    if (SINGLE_SHORTCUT && tp.single) {
        TileRef r;
        r.u = tp.u_lo;
        r.ti = tp.one;
        r.e0 = static_cast<long long>(bid + tp.single_skip) * tp.tile;
        return r;
    }
    __shared__ int s_u;
    const int tile = bid + tp.tile_lo;
    for (int u = tp.u_lo + threadIdx.x; u < tp.u_hi; u += NT) {
        const int a = __ldg(tp.prefix + u), b = __ldg(tp.prefix + u + 1);
        if (a <= tile && tile < b) s_u = u;
    }
    __syncthreads();
    const int lo = s_u;
    TileRef r;
    r.u = lo;
    const int4 *rec = reinterpret_cast<const int4 *>(tp.info + lo);
    const int4 a = __ldg(rec), b = __ldg(rec + 1);
    r.ti.dst_off = (static_cast<long long>(a.y) << 32) | static_cast<unsigned>(a.x);
    r.ti.numel = (static_cast<long long>(a.w) << 32) | static_cast<unsigned>(a.z);
    r.ti.ext = (static_cast<long long>(b.y) << 32) | static_cast<unsigned>(b.x);
    r.ti.flags = b.z;
    r.ti.pad_ = 0;
    r.e0 = static_cast<long long>(tile - __ldg(tp.prefix + lo)) * tp.tile;
    return r;
}

// ------------------------------------------------------------------ K1: fused pack + widen + weighted intra-group reduce
// P_g[off_u + e] = sum_{r in g} a_r * f32(x_r^(u)[e]), zero in the padding.
template <typename Tin, typename TT, int KB, bool EDGE>
__device__ __forceinline__ void k1_tile(const K1Params &p, const TileRef &t) {
    constexpr int VEC = Elem<Tin>::VEC;
    constexpr int TILE = Elem<Tin>::TILE;
    constexpr int ITERS = TILE / (NT * VEC);
    const int K = p.rt.K;
    const int T = p.tp.T;
    const bool aligned = t.ti.flags & FLAG_ALIGNED;
    long long e[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) e[it] = t.e0 + (it * NT + threadIdx.x) * VEC;

    float acc[ITERS][VEC];
    for (int kb = 0; kb < K; kb += KB) {
        uint4 raw[KB][ITERS];
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (kb + j < K) {
                const Tin *s = static_cast<const Tin *>(ldg_ptr(&p.ptrs[static_cast<size_t>(kb + j) * T + t.u]));
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    if (!EDGE || (aligned && e[it] + VEC <= t.ti.numel))
                        raw[j][it] = ld_stream(s + e[it]);
                    else
                        raw[j][it] = Elem<Tin>::gather(s, e[it], t.ti.numel);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (kb + j < K) {
                const float a = p.rt.coef[kb + j];
                const bool first = p.rt.first[kb + j];
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    float x[VEC];
                    Elem<Tin>::unpack(raw[j][it], x);
#pragma unroll
                    for (int c = 0; c < VEC; ++c)
                        acc[it][c] = first ? __fmul_rn(a, x[c]) : __fmaf_rn(a, x[c], acc[it][c]);
                }
                if (p.rt.last[kb + j]) {
                    void *d = p.transport[p.rt.gid[kb + j]];
#pragma unroll
                    for (int it = 0; it < ITERS; ++it) {
                        if (EDGE) {
                            if (e[it] >= t.ti.ext) continue;
#pragma unroll
                            for (int c = 0; c < VEC; ++c)   // padding is +0 whatever the weights
                                if (e[it] + c >= t.ti.numel) acc[it][c] = 0.f;
                        }
                        store_transport<TT, VEC>(d, t.ti.dst_off + e[it], acc[it], p.wide);
                    }
                }
            }
        }
    }
}

template <typename Tin, typename TT, int KB>
__global__ void __launch_bounds__(NT, 1024 / NT) k1_intra_reduce(const __grid_constant__ K1Params p) {
    const TileRef t = locate_tile<true>(p.tp);
    if ((t.ti.flags & FLAG_ALIGNED) && t.e0 + Elem<Tin>::TILE <= t.ti.numel)
        k1_tile<Tin, TT, KB, false>(p, t);
    else
        k1_tile<Tin, TT, KB, true>(p, t);
}

// ------------------------------------------------------------------ K2: inter-group combine + scale + cast + unpack
// out_c^(u)[e] = cast(scale * sum_g W_g P_g[off_u + e]) for every copy c < R.
template <typename Tout, typename TT, int TILE, bool EDGE>
__device__ __forceinline__ void k2_tile(const K2Params &p, const TileRef &t) {
    constexpr int VEC = Elem<Tout>::VEC;
    constexpr int ITERS = TILE / (NT * VEC);
    const int G = p.gt.G;
    const int T = p.tp.T;
    const bool aligned = p.out_aligned[t.u];
    // fp32 outputs: the destination of the first copy is fetched now, beside the partials, not
    // after them (measured: -5 % on large buckets; for bf16 outputs the extra live register
    // costs a resident CTA and the early fetch loses)
    constexpr bool EARLY_OUT = sizeof(Tout) == 4;
    Tout *first_out = nullptr;
    if (EARLY_OUT) first_out = static_cast<Tout *>(ldg_ptr(&p.out_ptrs[t.u]));
    long long e[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) e[it] = t.e0 + (it * NT + threadIdx.x) * VEC;

    float acc[ITERS][VEC];
    for (int g = 0; g < G; ++g) {
        const float w = p.gt.W[g];
        float x[ITERS][VEC];
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            // the transport holds ext elements per tensor, so a vector below ext is readable
            if (!EDGE || e[it] < t.ti.ext) {
                load_transport<TT, VEC>(p.src[g], t.ti.dst_off + e[it], x[it], p.wide);
            } else {
#pragma unroll
                for (int c = 0; c < VEC; ++c) x[it][c] = 0.f;
            }
        }
#pragma unroll
        for (int it = 0; it < ITERS; ++it)
#pragma unroll
            for (int c = 0; c < VEC; ++c)
                acc[it][c] = g == 0 ? __fmul_rn(w, x[it][c]) : __fmaf_rn(w, x[it][c], acc[it][c]);
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        float y[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) y[c] = __fmul_rn(acc[it][c], p.scale);
        if (!EDGE || (aligned && e[it] + VEC <= t.ti.numel)) {
            const uint4 o = Elem<Tout>::narrow(y);
            if (EARLY_OUT) *reinterpret_cast<uint4 *>(first_out + e[it]) = o;
            for (int c = EARLY_OUT ? 1 : 0; c < p.R; ++c)
                *reinterpret_cast<uint4 *>(static_cast<Tout *>(ldg_ptr(&p.out_ptrs[static_cast<size_t>(c) * T + t.u])) + e[it]) = o;
        } else if (e[it] < t.ti.numel) {
            for (int c = 0; c < p.R; ++c) {
                Tout *d = static_cast<Tout *>(ldg_ptr(&p.out_ptrs[static_cast<size_t>(c) * T + t.u]));
#pragma unroll
                for (int k = 0; k < VEC; ++k)
                    if (e[it] + k < t.ti.numel) d[e[it] + k] = Elem<Tout>::narrow_one(y[k]);
            }
        }
    }
}

// Five resident CTAs per SM (48 registers): measured 1.5-2.5 % faster than the compiler's own
// choice of 54-64 registers on fp32 outputs, equal on bf16 outputs; six (40 registers) lost.
template <typename Tout, typename TT, int TILE>
__global__ void __launch_bounds__(NT, 5) k2_combine_unpack(const __grid_constant__ K2Params p) {
    // Tiles are taken from the end of the range backwards: the partials were written front to
    // back just before (by the fused reduce, or by the copy up), so the end of the range is what
    // the L2 still holds; read front to back, the kernel's own traffic would have evicted it
    // before getting there (measured: -14 % on ResNet-50's 204 MB of partials, no change where
    // the partials fit the L2 whole).
    const TileRef t = locate_tile(p.tp, gridDim.x - 1 - blockIdx.x);
    if (p.out_aligned[t.u] && t.e0 + TILE <= t.ti.numel)
        k2_tile<Tout, TT, TILE, false>(p, t);
    else
        k2_tile<Tout, TT, TILE, true>(p, t);
}

// ------------------------------------------------------------------ direct path: reduce, combine, scale, cast, unpack in one pass
// Section III-B: a collective whose participants need no host relay is dispatched straight
// to the device-side reduction.  Same arithmetic and order as K1 followed by K2, with the
// group partials kept in registers instead of a transport buffer:
//   out_c^(u)[e] = cast(scale * sum_g W_g * (sum_{r in g} a_r * f32(x_r^(u)[e]))).
template <typename Tout, int VEC>
__device__ __forceinline__ void store_out(Tout *d, const float (&y)[VEC]) {
    if constexpr (sizeof(Tout) == 4) {
#pragma unroll
        for (int q = 0; q < VEC / 4; ++q)
            reinterpret_cast<float4 *>(d)[q] = make_float4(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
    } else if constexpr (VEC == 8) {
        *reinterpret_cast<uint4 *>(d) = make_uint4(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]),
                                                   pack_bf16x2(y[4], y[5]), pack_bf16x2(y[6], y[7]));
    } else {
        *reinterpret_cast<uint2 *>(d) = make_uint2(pack_bf16x2(y[0], y[1]), pack_bf16x2(y[2], y[3]));
    }
}

// INPLACE: some output tensor is one of the registered gradient tensors (an all-reduce in
// place).  Every thread reads all ranks' values of its elements before it writes them, so the
// result is the same; only the loads must not take the read-only path.
template <typename Tin, typename Tout, int KB, bool EDGE, bool INPLACE>
__device__ __forceinline__ void direct_tile(const DirectParams &p, const TileRef &t) {
    constexpr int VEC = Elem<Tin>::VEC;
    constexpr int TILE = Elem<Tin>::TILE;
    constexpr int ITERS = TILE / (NT * VEC);
    const int K = p.rt.K;
    const int T = p.tp.T;
    const bool aligned = t.ti.flags & FLAG_ALIGNED;
    long long e[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) e[it] = t.e0 + (it * NT + threadIdx.x) * VEC;

    float acc[ITERS][VEC], sum[ITERS][VEC];
    for (int kb = 0; kb < K; kb += KB) {
        uint4 raw[KB][ITERS];
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (kb + j < K) {
                const Tin *s = static_cast<const Tin *>(ldg_ptr(&p.ptrs[static_cast<size_t>(kb + j) * T + t.u]));
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    if (!EDGE || (aligned && e[it] + VEC <= t.ti.numel))
                        raw[j][it] = INPLACE ? ld_plain(s + e[it]) : ld_stream(s + e[it]);
                    else
                        raw[j][it] = Elem<Tin>::gather(s, e[it], t.ti.numel);
                }
            }
        }
#pragma unroll
        for (int j = 0; j < KB; ++j) {
            if (kb + j < K) {
                const float a = p.rt.coef[kb + j];
                const bool first = p.rt.first[kb + j];
#pragma unroll
                for (int it = 0; it < ITERS; ++it) {
                    float x[VEC];
                    Elem<Tin>::unpack(raw[j][it], x);
#pragma unroll
                    for (int c = 0; c < VEC; ++c)
                        acc[it][c] = first ? __fmul_rn(a, x[c]) : __fmaf_rn(a, x[c], acc[it][c]);
                }
                if (p.rt.last[kb + j]) {           // the group's partial is complete: fold it in
                    const int g = p.rt.gid[kb + j];
                    const float w = p.gt.W[g];
#pragma unroll
                    for (int it = 0; it < ITERS; ++it)
#pragma unroll
                        for (int c = 0; c < VEC; ++c)
                            sum[it][c] = g == 0 ? __fmul_rn(w, acc[it][c]) : __fmaf_rn(w, acc[it][c], sum[it][c]);
                }
            }
        }
    }
    const bool out_aligned = p.out_aligned[t.u];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        float y[VEC];
#pragma unroll
        for (int c = 0; c < VEC; ++c) y[c] = __fmul_rn(sum[it][c], p.scale);
        if (!EDGE || (out_aligned && e[it] + VEC <= t.ti.numel)) {
            for (int c = 0; c < p.R; ++c)
                store_out<Tout, VEC>(static_cast<Tout *>(ldg_ptr(&p.out_ptrs[static_cast<size_t>(c) * T + t.u])) + e[it], y);
        } else if (e[it] < t.ti.numel) {
            for (int c = 0; c < p.R; ++c) {
                Tout *d = static_cast<Tout *>(ldg_ptr(&p.out_ptrs[static_cast<size_t>(c) * T + t.u]));
#pragma unroll
                for (int k = 0; k < VEC; ++k)
                    if (e[it] + k < t.ti.numel) d[e[it] + k] = Elem<Tout>::narrow_one(y[k]);
            }
        }
    }
}

template <typename Tin, typename Tout, int KB, bool INPLACE>
__global__ void __launch_bounds__(NT) k_direct_sync(const __grid_constant__ DirectParams p) {
    const TileRef t = locate_tile(p.tp);
    if ((t.ti.flags & FLAG_ALIGNED) && p.out_aligned[t.u] && t.e0 + Elem<Tin>::TILE <= t.ti.numel)
        direct_tile<Tin, Tout, KB, false, INPLACE>(p, t);
    else
        direct_tile<Tin, Tout, KB, true, INPLACE>(p, t);
}

// ------------------------------------------------------------------ flat inter-group combine into a combined buffer
template <typename TT>
__global__ void __launch_bounds__(NT) k_combine_flat(const __grid_constant__ K2Params p, float *combined,
                                                     long long lo, long long n4) {
    const int G = p.gt.G;
    for (long long i = blockIdx.x * static_cast<long long>(NT) + threadIdx.x; i < n4;
         i += static_cast<long long>(gridDim.x) * NT) {
        const long long e = lo + 4 * i;
        float acc[4];
        for (int g = 0; g < G; ++g) {
            float x[4];
            load_transport<TT, 4>(p.src[g], e, x, false);
            const float w = p.gt.W[g];
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[c] = g == 0 ? __fmul_rn(w, x[c]) : __fmaf_rn(w, x[c], acc[c]);
        }
        *reinterpret_cast<float4 *>(combined + e) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    }
}

// ------------------------------------------------------------------ standalone pack (bit copy of every rank's tensors into its flat buffer)
template <typename Tin>
__global__ void __launch_bounds__(NT) k_pack(const __grid_constant__ PackParams p) {
    constexpr int VEC = Elem<Tin>::VEC;
    constexpr int TILE = Elem<Tin>::TILE;
    constexpr int ITERS = TILE / (NT * VEC);
    const TileRef t = locate_tile(p.tp);
    const int k = blockIdx.y;
    const Tin *s = static_cast<const Tin *>(ldg_ptr(&p.ptrs[static_cast<size_t>(k) * p.tp.T + t.u]));
    Tin *flat = static_cast<Tin *>(p.flat[k]) + t.ti.dst_off;
    const bool aligned = t.ti.flags & FLAG_ALIGNED;
    uint4 raw[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const long long e = t.e0 + (it * NT + threadIdx.x) * VEC;
        if (aligned && e + VEC <= t.ti.numel) raw[it] = ld_stream(s + e);
        else raw[it] = Elem<Tin>::gather(s, e, t.ti.numel);
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        const long long e = t.e0 + (it * NT + threadIdx.x) * VEC;
        // ext is a multiple of 8 elements, so a vector that starts below ext ends inside it
        if (e < t.ti.ext) *reinterpret_cast<uint4 *>(flat + e) = raw[it];
    }
}

// ------------------------------------------------------------------ hierarchical broadcast (model synchronisation)
// Section III-A routes Broadcast like AllReduce: inside the root's group directly, to the
// other groups through host RAM.  Both kernels are bit copies.
//
// element c of a 16-byte vector written to d[c] for the elements below n (tails, misaligned tensors)
template <typename Tv>
__device__ __forceinline__ void store_elems(Tv *d, const uint4 &v, long long e, long long n) {
    const unsigned w[4] = {v.x, v.y, v.z, v.w};
    constexpr int VEC = Elem<Tv>::VEC;
#pragma unroll
    for (int c = 0; c < VEC; ++c) {
        if (e + c >= n) break;
        if constexpr (sizeof(Tv) == 4) d[e + c] = __uint_as_float(w[c]);
        else d[e + c] = static_cast<unsigned short>(w[c / 2] >> (16 * (c & 1)));
    }
}

// send side: the root's tensors are read once; every element goes to the flat send buffer of
// the root's group (plan offsets, zero padding) and to the tensors of the root's group mates
template <typename Tv>
__global__ void __launch_bounds__(NT) k_bcast_send(const __grid_constant__ BcastParams p) {
    constexpr int VEC = Elem<Tv>::VEC;
    constexpr int ITERS = Elem<Tv>::TILE / (NT * VEC);
    const TileRef t = locate_tile(p.tp);
    const int T = p.tp.T;
    const Tv *s = static_cast<const Tv *>(ldg_ptr(&p.ptrs[static_cast<size_t>(p.k_root) * T + t.u]));
    Tv *flat = static_cast<Tv *>(p.flat[p.g_root]) + t.ti.dst_off;
    const bool aligned = t.ti.flags & FLAG_ALIGNED;
    uint4 raw[ITERS];
    long long e[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
        e[it] = t.e0 + (it * NT + threadIdx.x) * VEC;
        if (aligned && e[it] + VEC <= t.ti.numel) raw[it] = ld_stream(s + e[it]);
        else raw[it] = Elem<Tv>::gather(s, e[it], t.ti.numel);
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it)
        if (e[it] < t.ti.ext) *reinterpret_cast<uint4 *>(flat + e[it]) = raw[it];
    for (int k = p.k_lo[p.g_root]; k < p.k_hi[p.g_root]; ++k) {
        if (k == p.k_root) continue;
        Tv *d = static_cast<Tv *>(ldg_ptr(&p.ptrs[static_cast<size_t>(k) * T + t.u]));
#pragma unroll
        for (int it = 0; it < ITERS; ++it) {
            if (aligned && e[it] + VEC <= t.ti.numel) *reinterpret_cast<uint4 *>(d + e[it]) = raw[it];
            else store_elems<Tv>(d, raw[it], e[it], t.ti.numel);
        }
    }
}

// receive side: every other group reads its own flat receive buffer once and writes the
// tensors of all its members
template <typename Tv>
__global__ void __launch_bounds__(NT) k_bcast_recv(const __grid_constant__ BcastParams p) {
    constexpr int VEC = Elem<Tv>::VEC;
    constexpr int ITERS = Elem<Tv>::TILE / (NT * VEC);
    const TileRef t = locate_tile(p.tp);
    const int T = p.tp.T;
    const bool aligned = t.ti.flags & FLAG_ALIGNED;
    long long e[ITERS];
#pragma unroll
    for (int it = 0; it < ITERS; ++it) e[it] = t.e0 + (it * NT + threadIdx.x) * VEC;
    for (int g = 0; g < p.G; ++g) {
        if (g == p.g_root) continue;
        const Tv *s = static_cast<const Tv *>(p.flat[g]) + t.ti.dst_off;
        uint4 raw[ITERS];
#pragma unroll
        for (int it = 0; it < ITERS; ++it)   // ext is a multiple of 8 elements: a vector below ext is readable
            raw[it] = e[it] < t.ti.ext ? ld_stream(s + e[it]) : make_uint4(0u, 0u, 0u, 0u);
        for (int k = p.k_lo[g]; k < p.k_hi[g]; ++k) {
            Tv *d = static_cast<Tv *>(ldg_ptr(&p.ptrs[static_cast<size_t>(k) * T + t.u]));
#pragma unroll
            for (int it = 0; it < ITERS; ++it) {
                if (aligned && e[it] + VEC <= t.ti.numel) *reinterpret_cast<uint4 *>(d + e[it]) = raw[it];
                else store_elems<Tv>(d, raw[it], e[it], t.ti.numel);
            }
        }
    }
}

// ------------------------------------------------------------------ load-adaptive sampler (Section III-C, dynamic data allocation)
// Position p of the epoch's index list belongs to step s = p / B; inside the step rank r owns
// the b_r positions from c_r on.  out_r[s * b_r + j] = list[(s * B + c_r + j) mod D].
struct SamplerParams {
    const long long *list;              // epoch permutation (device) or NULL for the identity
    long long D;                        // dataset size
    long long total;                    // S * B positions
    int B, K;
    int start[KT_MAX_RANKS + 1];        // c_r, start[K] = B
    long long *out[KT_MAX_RANKS];
};

__global__ void __launch_bounds__(NT) k_sampler(const __grid_constant__ SamplerParams p) {
    for (long long pos = blockIdx.x * static_cast<long long>(NT) + threadIdx.x; pos < p.total;
         pos += static_cast<long long>(gridDim.x) * NT) {
        const long long step = pos / p.B;
        const int w = static_cast<int>(pos - step * p.B);
        int lo = 0, hi = p.K;                           // rank with start[r] <= w < start[r + 1]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (p.start[mid] <= w) lo = mid; else hi = mid;
        }
        const long long src = pos % p.D;
        const long long v = p.list ? __ldg(p.list + src) : src;
        const int b = p.start[lo + 1] - p.start[lo];
        p.out[lo][step * b + (w - p.start[lo])] = v;
    }
}

// ------------------------------------------------------------------ standalone casts
__global__ void __launch_bounds__(NT) k_cast_bf16_to_f32(const unsigned short *in, float *out, long long n) {
    for (long long i = blockIdx.x * static_cast<long long>(NT) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * NT)
        out[i] = __uint_as_float(static_cast<unsigned>(in[i]) << 16);
}
__global__ void __launch_bounds__(NT) k_cast_f32_to_bf16(const float *in, unsigned short *out, long long n) {
    for (long long i = blockIdx.x * static_cast<long long>(NT) + threadIdx.x; i < n;
         i += static_cast<long long>(gridDim.x) * NT)
        out[i] = static_cast<unsigned short>(pack_bf16x2(in[i], 0.f) & 0xFFFFu);
}

}  // namespace
