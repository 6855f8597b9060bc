// Device code of the SSD-SGD update path for sm_100a.
//
// Three streaming kernels sweep the flat parameter arena once per call:
//   sync_kernel   server: K-way gradient sum + momentum-SGD (+ the hand-over copy
//                 of the last warm-up iteration)
//   glu_kernel    one worker's GLU update (+ pre_weight refresh, + pull)
//   step_kernel   both of the above for all K workers in one pass: each gradient
//                 element is read once and feeds the server sum and its own
//                 worker's GLU update
// All three are bound by HBM bandwidth (well under one flop per byte), so the
// design is about bytes: 128-bit loads and stores, every byte touched once,
// streaming cache hints, several independent loads in flight per thread.
//
// Arithmetic contract: binary32, round to nearest, every operation rounded on
// its own.  The __f*_rn intrinsics are never contracted into fused multiply-adds,
// whatever the compiler flags.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ssd {

constexpr int kMaxWorkers = 32;
constexpr int kMaxThreads = 512;   // upper bound of threads per block for every kernel here

enum : int { kFirst = 1, kRefresh = 2, kPull = 4, kCopy = 8 };
enum : int { kF32 = 0, kBF16 = 1 };

struct Scalars {
    float lr, m, wd, rescale;      // server
    float lr_loc, alpha, beta, c;  // GLU; c = (1-m)/(lr*k)
};

struct SyncParams {
    const void *g[kMaxWorkers];
    float *w_loc[kMaxWorkers];     // written when flags has kCopy
    float *w, *mom;
    int64_t n;
    int K, flags;
    Scalars s;
};

struct GluParams {
    const void *g;
    float *w_loc, *pre, *w_dev;
    const float *w;                // read when flags has kPull
    int64_t n;
    int flags;
    Scalars s;
};

struct StepParams {
    const void *g[kMaxWorkers];
    float *w_loc[kMaxWorkers];
    float *pre[kMaxWorkers];
    float *w_dev[kMaxWorkers];
    float *w, *mom;
    int64_t n;
    int K, flags;
    Scalars s;
};

struct CopyParams {
    float *dst[kMaxWorkers];
    const float *src;
    int64_t n;
    int K;
};

// ---------------------------------------------------------------------------
// VW consecutive elements; VW = 4 is one 128-bit access.  Arena lengths are
// multiples of 4 elements by construction, so there is no ragged tail.
// ---------------------------------------------------------------------------
template <int VW> struct Vec { float v[VW]; };

template <int VW> __device__ __forceinline__ Vec<VW> ld_f32(const float *p, int64_t e);
template <> __device__ __forceinline__ Vec<4> ld_f32<4>(const float *p, int64_t e)
{
    float4 t = __ldcs(reinterpret_cast<const float4 *>(p + e));
    return Vec<4>{{t.x, t.y, t.z, t.w}};
}

template <int VW> __device__ __forceinline__ void st_f32(float *p, int64_t e, const Vec<VW> &x);
template <> __device__ __forceinline__ void st_f32<4>(float *p, int64_t e, const Vec<4> &x)
{
    __stcs(reinterpret_cast<float4 *>(p + e), make_float4(x.v[0], x.v[1], x.v[2], x.v[3]));
}

__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

// Gradient load: float32 as is, bfloat16 widened exactly (bits << 16).
template <int GT, int VW> __device__ __forceinline__ Vec<VW> ld_grad(const void *p, int64_t e);
template <> __device__ __forceinline__ Vec<4> ld_grad<kF32, 4>(const void *p, int64_t e)
{
    return ld_f32<4>(static_cast<const float *>(p), e);
}
template <> __device__ __forceinline__ Vec<4> ld_grad<kBF16, 4>(const void *p, int64_t e)
{
    uint2 t = __ldcs(reinterpret_cast<const uint2 *>(static_cast<const uint16_t *>(p) + e));
    return Vec<4>{{bf16_lo(t.x), bf16_hi(t.x), bf16_lo(t.y), bf16_hi(t.y)}};
}

// ---------------------------------------------------------------------------
// Per-element arithmetic.
// ---------------------------------------------------------------------------

// Server momentum-SGD (Section 3.2.1): mom = m*mom - lr*(grad + wd*w); w = w + mom,
// with grad = (left-to-right sum of the K gradients) * rescale.
__device__ __forceinline__ void server_elem(float gsum, float &w, float &mom, const Scalars &s)
{
    float grad = __fmul_rn(gsum, s.rescale);
    float full = __fadd_rn(grad, __fmul_rn(s.wd, w));
    float step = __fmul_rn(s.lr, full);
    float keep = __fmul_rn(s.m, mom);
    mom = __fsub_rn(keep, step);
    w = __fadd_rn(w, mom);
}

// GLU rule with grad_sync = (pre_weight - w')*c (Section 3.3):
//   w' - lr_loc*((alpha*g + wd*w') + beta*grad_sync)
__device__ __forceinline__ float glu_elem(float g, float wl, float pre, const Scalars &s)
{
    float gs = __fmul_rn(__fsub_rn(pre, wl), s.c);
    float mix = __fadd_rn(__fmul_rn(s.alpha, g), __fmul_rn(s.wd, wl));
    mix = __fadd_rn(mix, __fmul_rn(s.beta, gs));
    return __fsub_rn(wl, __fmul_rn(s.lr_loc, mix));
}

// ---------------------------------------------------------------------------
// Bodies, written once for a vector of VW elements at element offset e.
// B = workers whose loads are issued together before any is consumed.
// ---------------------------------------------------------------------------

template <int GT, int VW, int B>
__device__ __forceinline__ void sync_at(const SyncParams &p, int64_t e)
{
    Vec<VW> w = ld_f32<VW>(p.w, e);
    Vec<VW> mom = ld_f32<VW>(p.mom, e);
    Vec<VW> sum;
    for (int i0 = 0; i0 < p.K; i0 += B) {
        Vec<VW> g[B];
#pragma unroll
        for (int b = 0; b < B; ++b)
            if (i0 + b < p.K) g[b] = ld_grad<GT, VW>(p.g[i0 + b], e);
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (i0 + b < p.K) {
#pragma unroll
                for (int l = 0; l < VW; ++l)
                    sum.v[l] = (i0 + b == 0) ? g[b].v[l] : __fadd_rn(sum.v[l], g[b].v[l]);
            }
        }
    }
#pragma unroll
    for (int l = 0; l < VW; ++l) server_elem(sum.v[l], w.v[l], mom.v[l], p.s);
    st_f32<VW>(p.mom, e, mom);
    st_f32<VW>(p.w, e, w);
    if (p.flags & kCopy)
        for (int i = 0; i < p.K; ++i) st_f32<VW>(p.w_loc[i], e, w);
}

template <int GT, int VW>
__device__ __forceinline__ void glu_at(const GluParams &p, int64_t e)
{
    const bool first = p.flags & kFirst, refresh = p.flags & kRefresh, pull = p.flags & kPull;
    Vec<VW> g = ld_grad<GT, VW>(p.g, e);
    Vec<VW> wl = ld_f32<VW>(p.w_loc, e);
    Vec<VW> pr = first ? wl : ld_f32<VW>(p.pre, e);
    Vec<VW> wg;
    if (pull) wg = ld_f32<VW>(p.w, e);
    Vec<VW> r;
#pragma unroll
    for (int l = 0; l < VW; ++l) r.v[l] = glu_elem(g.v[l], wl.v[l], pr.v[l], p.s);
    if (first || refresh) st_f32<VW>(p.pre, e, wl);
    if (pull) {
        st_f32<VW>(p.w_dev, e, r);
        st_f32<VW>(p.w_loc, e, wg);
    } else {
        st_f32<VW>(p.w_loc, e, r);
    }
}

template <int GT, int VW, int B>
__device__ __forceinline__ void step_at(const StepParams &p, int64_t e)
{
    const bool first = p.flags & kFirst, refresh = p.flags & kRefresh, pull = p.flags & kPull;
    Vec<VW> w = ld_f32<VW>(p.w, e);
    Vec<VW> mom = ld_f32<VW>(p.mom, e);
    Vec<VW> sum;
    for (int i0 = 0; i0 < p.K; i0 += B) {
        Vec<VW> g[B], wl[B], pr[B];
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (i0 + b < p.K) {
                g[b] = ld_grad<GT, VW>(p.g[i0 + b], e);
                wl[b] = ld_f32<VW>(p.w_loc[i0 + b], e);
                if (!first) pr[b] = ld_f32<VW>(p.pre[i0 + b], e);
            }
        }
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (i0 + b < p.K) {
                const int i = i0 + b;
                Vec<VW> r;
#pragma unroll
                for (int l = 0; l < VW; ++l) {
                    sum.v[l] = (i == 0) ? g[b].v[l] : __fadd_rn(sum.v[l], g[b].v[l]);
                    r.v[l] = glu_elem(g[b].v[l], wl[b].v[l], first ? wl[b].v[l] : pr[b].v[l], p.s);
                }
                if (first || refresh) st_f32<VW>(p.pre[i], e, wl[b]);
                st_f32<VW>(pull ? p.w_dev[i] : p.w_loc[i], e, r);
            }
        }
    }
#pragma unroll
    for (int l = 0; l < VW; ++l) server_elem(sum.v[l], w.v[l], mom.v[l], p.s);
    st_f32<VW>(p.mom, e, mom);
    st_f32<VW>(p.w, e, w);
    if (pull)
        for (int i = 0; i < p.K; ++i) st_f32<VW>(p.w_loc[i], e, w);
}

// ---------------------------------------------------------------------------
// Kernels: grid-stride over the n/4 128-bit vectors of the arena.
// ---------------------------------------------------------------------------
#define SSD_SWEEP(n, BODY)                                                                \
    do {                                                                                  \
        const int64_t nvec = (n) >> 2;                                                    \
        const int64_t stride = (int64_t)gridDim.x * blockDim.x;                           \
        for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) { \
            const int64_t e = v << 2;                                                     \
            BODY;                                                                         \
        }                                                                                 \
    } while (0)

template <int GT, int B>
__global__ void __launch_bounds__(kMaxThreads) sync_kernel(const __grid_constant__ SyncParams p)
{
    SSD_SWEEP(p.n, (sync_at<GT, 4, B>(p, e)));
}

template <int GT>
__global__ void __launch_bounds__(kMaxThreads) glu_kernel(const __grid_constant__ GluParams p)
{
    SSD_SWEEP(p.n, (glu_at<GT, 4>(p, e)));
}

template <int GT, int B>
__global__ void __launch_bounds__(kMaxThreads) step_kernel(const __grid_constant__ StepParams p)
{
    SSD_SWEEP(p.n, (step_at<GT, 4, B>(p, e)));
}

// dst[i] = src for K destinations (the pull of a freshly initialised or warm-up weight).
__global__ void __launch_bounds__(kMaxThreads) copy_kernel(const __grid_constant__ CopyParams p)
{
    SSD_SWEEP(p.n, {
        Vec<4> x = ld_f32<4>(p.src, e);
        for (int i = 0; i < p.K; ++i) st_f32<4>(p.dst[i], e, x);
    });
}

}  // namespace ssd
