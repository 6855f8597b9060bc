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
// design is about bytes: every byte touched once, 256-bit (or 128-bit) fully
// coalesced accesses, streaming cache hints, and enough independent loads in
// flight per SM to cover the DRAM latency.
//
// Arithmetic contract: binary32, round to nearest, every operation rounded on
// its own.  The __f*_rn intrinsics are never contracted into fused multiply-adds,
// whatever the compiler flags.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

// Cache policy of the streaming accesses: state and gradients are far larger than L2 and each
// byte is used once per kernel, so every load and store carries the evict-first hint (.cs).
// Measured against the default policy, .cg and .nc on B200 the differences stayed within 2 %.
namespace ssd {

constexpr int kMaxWorkers = 32;
constexpr int kMaxThreads = 512;   // upper bound of threads per block for every kernel here

// kLocalSgd, kMergedDev: internal.  kMergedDev: the workers' device weights are the same buffers as
// their local weights, so on a pull iteration the local update's result has nowhere to go (the
// pulled global weight overwrites it at once) and is neither computed nor stored; such iterations
// run the *_merged_pull kernels instead of glu_kernel / step_kernel.
enum : int { kFirst = 1, kRefresh = 2, kPull = 4, kCopy = 8, kLocalSgd = 16, kMergedDev = 32 };
enum : int { kF32 = 0, kBF16 = 1 };

struct Scalars {
    float lr, m, wd, rescale;      // server
    float lr_loc, alpha, beta, c;  // GLU; c = (1-m)/(lr*k)
};

// Optional per-tensor scalars (device memory, filled by the host): tensor t covers arena
// positions [end[t-1], end[t]) and uses scal[t] = {lr, wd, lr_loc, c} instead of the uniform
// values in Scalars.  T == 0: uniform.
struct TensorTable {
    const int64_t *end;
    const float4 *scal;
    int64_t base;                  // arena position of the launch's element 0 (range launches)
    int T;
};

struct SyncParams {
    const void *g[kMaxWorkers];
    float *w_loc[kMaxWorkers];     // written when flags has kCopy
    float *w, *mom;
    int64_t n;
    int K, flags;
    int per_batch;                 // workers per batch of loads: K split evenly over ceil(K / B) batches
    Scalars s;
    TensorTable tt;
};

struct GluParams {
    const void *g;
    float *w_loc, *pre, *w_dev;
    const float *w;                // read when flags has kPull
    int64_t n;
    int flags;
    Scalars s;
    TensorTable tt;
};

struct StepParams {
    const void *g[kMaxWorkers];
    float *w_loc[kMaxWorkers];
    float *pre[kMaxWorkers];
    float *w_dev[kMaxWorkers];
    float *w, *mom;
    int64_t n;
    int K, flags;
    int per_batch;                 // workers per batch of loads: K split evenly over ceil(K / B) batches
    int shared_pre;                // 1: pre[0] is the one pre_weight of all workers
    Scalars s;
    TensorTable tt;
};

struct CopyParams {
    float *dst[kMaxWorkers];
    const float *src;
    int64_t n;
    int K;
};

// ---------------------------------------------------------------------------
// VW consecutive elements owned by one thread: VW = 8 is one 256-bit access to
// float32 data (sm_100 has 256-bit global loads and stores) and one 128-bit
// access to bfloat16 data; VW = 16 is two adjacent 256-bit accesses to float32
// data and ONE 256-bit access to bfloat16 data, so that bfloat16 gradients are
// fetched with the widest load too; VW = 4 is the 128-bit / 64-bit form for
// buffers that are only 16-byte aligned, and finishes a length that is not a
// multiple of VW.
// ---------------------------------------------------------------------------
template <int VW> struct Vec { float v[VW]; };

// Loads of VW float32 values with a given cache qualifier.
#define SSD_DEFINE_LD_F32(NAME, QUAL)                                                           \
    template <int VW> __device__ __forceinline__ Vec<VW> NAME(const float *p, int64_t e);       \
    template <> __device__ __forceinline__ Vec<4> NAME<4>(const float *p, int64_t e)            \
    {                                                                                           \
        Vec<4> r;                                                                               \
        asm volatile("ld.global" QUAL ".v4.f32 {%0,%1,%2,%3}, [%4];"                            \
                     : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3])                   \
                     : "l"(p + e));                                                             \
        return r;                                                                               \
    }                                                                                           \
    template <> __device__ __forceinline__ Vec<8> NAME<8>(const float *p, int64_t e)            \
    {                                                                                           \
        Vec<8> r;                                                                               \
        asm volatile("ld.global" QUAL ".v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"                \
                     : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]),    \
                       "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])                                 \
                     : "l"(p + e));                                                             \
        return r;                                                                               \
    }                                                                                           \
    template <> __device__ __forceinline__ Vec<16> NAME<16>(const float *p, int64_t e)          \
    {                                                                                           \
        const Vec<8> a = NAME<8>(p, e), b = NAME<8>(p, e + 8);                                  \
        Vec<16> r;                                                                              \
        _Pragma("unroll") for (int l = 0; l < 8; ++l) { r.v[l] = a.v[l]; r.v[8 + l] = b.v[l]; } \
        return r;                                                                               \
    }

SSD_DEFINE_LD_F32(ld_f32, ".cs")        // state: read, then overwritten by the same thread
SSD_DEFINE_LD_F32(ld_f32_ro, ".cs")    // gradients: read-only for the whole kernel

template <int VW> __device__ __forceinline__ void st_f32(float *p, int64_t e, const Vec<VW> &x);
template <> __device__ __forceinline__ void st_f32<4>(float *p, int64_t e, const Vec<4> &x)
{
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p + e), "f"(x.v[0]),
                 "f"(x.v[1]), "f"(x.v[2]), "f"(x.v[3])
                 : "memory");
}
template <> __device__ __forceinline__ void st_f32<8>(float *p, int64_t e, const Vec<8> &x)
{
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p + e),
                 "f"(x.v[0]), "f"(x.v[1]), "f"(x.v[2]), "f"(x.v[3]), "f"(x.v[4]), "f"(x.v[5]),
                 "f"(x.v[6]), "f"(x.v[7])
                 : "memory");
}

template <> __device__ __forceinline__ void st_f32<16>(float *p, int64_t e, const Vec<16> &x)
{
    Vec<8> a, b;
#pragma unroll
    for (int l = 0; l < 8; ++l) { a.v[l] = x.v[l]; b.v[l] = x.v[8 + l]; }
    st_f32<8>(p, e, a);
    st_f32<8>(p, e + 8, b);
}

__device__ __forceinline__ float bf16_lo(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }

// A gradient vector as loaded: float32 values, or bfloat16 kept packed two per
// register until they are used (a load in flight then costs one register per four
// bytes for either type).  get(l) widens bfloat16 exactly (bits << 16).
template <int GT, int VW> struct Grad;
template <int VW> struct Grad<kF32, VW> {
    Vec<VW> raw;
    __device__ __forceinline__ float get(int l) const { return raw.v[l]; }
};
template <int VW> struct Grad<kBF16, VW> {
    uint32_t raw[VW / 2];
    __device__ __forceinline__ float get(int l) const
    {
        return (l & 1) ? bf16_hi(raw[l >> 1]) : bf16_lo(raw[l >> 1]);
    }
};

template <int GT, int VW> __device__ __forceinline__ Grad<GT, VW> ld_grad(const void *p, int64_t e);
template <> __device__ __forceinline__ Grad<kF32, 4> ld_grad<kF32, 4>(const void *p, int64_t e)
{
    return Grad<kF32, 4>{ld_f32_ro<4>(static_cast<const float *>(p), e)};
}
template <> __device__ __forceinline__ Grad<kF32, 8> ld_grad<kF32, 8>(const void *p, int64_t e)
{
    return Grad<kF32, 8>{ld_f32_ro<8>(static_cast<const float *>(p), e)};
}
template <> __device__ __forceinline__ Grad<kF32, 16> ld_grad<kF32, 16>(const void *p, int64_t e)
{
    return Grad<kF32, 16>{ld_f32_ro<16>(static_cast<const float *>(p), e)};
}
template <> __device__ __forceinline__ Grad<kBF16, 4> ld_grad<kBF16, 4>(const void *p, int64_t e)
{
    Grad<kBF16, 4> r;
    asm volatile("ld.global.cs.v2.u32 {%0,%1}, [%2];"
                 : "=r"(r.raw[0]), "=r"(r.raw[1])
                 : "l"(static_cast<const uint16_t *>(p) + e));
    return r;
}
template <> __device__ __forceinline__ Grad<kBF16, 8> ld_grad<kBF16, 8>(const void *p, int64_t e)
{
    Grad<kBF16, 8> r;
    asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.raw[0]), "=r"(r.raw[1]), "=r"(r.raw[2]), "=r"(r.raw[3])
                 : "l"(static_cast<const uint16_t *>(p) + e));
    return r;
}

template <> __device__ __forceinline__ Grad<kBF16, 16> ld_grad<kBF16, 16>(const void *p, int64_t e)
{
    Grad<kBF16, 16> r;
    asm volatile("ld.global.cs.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.raw[0]), "=r"(r.raw[1]), "=r"(r.raw[2]), "=r"(r.raw[3]), "=r"(r.raw[4]),
                   "=r"(r.raw[5]), "=r"(r.raw[6]), "=r"(r.raw[7])
                 : "l"(static_cast<const uint16_t *>(p) + e));
    return r;
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

// Plain SGD as local updater (Eq. 5 with the descent sign): w' - lr_loc*(g + wd*w').
__device__ __forceinline__ float local_sgd_elem(float g, float wl, const Scalars &s)
{
    return __fsub_rn(wl, __fmul_rn(s.lr_loc, __fadd_rn(g, __fmul_rn(s.wd, wl))));
}

// ---------------------------------------------------------------------------
// Per-tensor scalars.  Tensors start on multiples of 4 elements, so each group of
// 4 consecutive elements lies in one tensor; a vector of 8 may straddle two.  The
// search runs after the thread's loads have been issued, under their latency.
// ---------------------------------------------------------------------------
__device__ __forceinline__ int tensor_of(const TensorTable &tt, int64_t e)
{
    int lo = 0, hi = tt.T - 1;                 // first t with end[t] > e
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(tt.end + mid) > e) hi = mid; else lo = mid + 1;
    }
    return lo;
}

__device__ __forceinline__ Scalars with_tensor(Scalars s, const TensorTable &tt, int t)
{
    const float4 v = __ldg(tt.scal + t);
    s.lr = v.x; s.wd = v.y; s.lr_loc = v.z; s.c = v.w;
    return s;
}

// Scalars of each 4-element group of the vector at element offset e.
template <bool PT, int VW> struct GroupScalars {
    Scalars g[VW / 4];
    __device__ __forceinline__ GroupScalars(const Scalars &uniform, const TensorTable &tt, int64_t e)
    {
#pragma unroll
        for (int q = 0; q < VW / 4; ++q) g[q] = uniform;
        if (PT) {
            const int64_t pos = e + tt.base;
            int t = tensor_of(tt, pos);
            int64_t tensor_end = __ldg(tt.end + t);
            g[0] = with_tensor(uniform, tt, t);
#pragma unroll
            for (int q = 1; q < VW / 4; ++q) {
                if (pos + 4 * q < tensor_end) {
                    g[q] = g[q - 1];
                } else {                       // the group starts in a later tensor
                    t = tensor_of(tt, pos + 4 * q);
                    tensor_end = __ldg(tt.end + t);
                    g[q] = with_tensor(uniform, tt, t);
                }
            }
        }
    }
    __device__ __forceinline__ const Scalars &at(int l) const { return g[l >> 2]; }
};

// ---------------------------------------------------------------------------
// Bodies, written once for a vector of VW elements at element offset e.
// B = workers whose loads are issued together before any is consumed.
// ---------------------------------------------------------------------------

template <int GT, int VW, int B, bool PT>
__device__ __forceinline__ void sync_at(const SyncParams &p, int64_t e)
{
    Vec<VW> w = ld_f32<VW>(p.w, e);
    Vec<VW> mom = ld_f32<VW>(p.mom, e);
    Vec<VW> sum;
    // batches of at most B workers, all of (nearly) the same size: 9 workers with B = 8 go as 5 + 4
    const int per = p.per_batch;
    for (int i0 = 0; i0 < p.K; i0 += per) {
        Grad<GT, VW> g[B];
#pragma unroll
        for (int b = 0; b < B; ++b)
            if (b < per && i0 + b < p.K) g[b] = ld_grad<GT, VW>(p.g[i0 + b], e);
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (b < per && i0 + b < p.K) {
#pragma unroll
                for (int l = 0; l < VW; ++l)
                    sum.v[l] = (i0 + b == 0) ? g[b].get(l) : __fadd_rn(sum.v[l], g[b].get(l));
            }
        }
    }
    const GroupScalars<PT, VW> sc(p.s, p.tt, e);
#pragma unroll
    for (int l = 0; l < VW; ++l) server_elem(sum.v[l], w.v[l], mom.v[l], sc.at(l));
    st_f32<VW>(p.mom, e, mom);
    st_f32<VW>(p.w, e, w);
    if (p.flags & kCopy)
        for (int i = 0; i < p.K; ++i) st_f32<VW>(p.w_loc[i], e, w);
}

template <int GT, int VW, bool PT>
__device__ __forceinline__ void glu_at(const GluParams &p, int64_t e)
{
    const bool sgd = p.flags & kLocalSgd;      // plain-SGD updater: pre_weight is not involved at all
    const bool first = (p.flags & kFirst) && !sgd, refresh = (p.flags & kRefresh) && !sgd, pull = p.flags & kPull;
    Grad<GT, VW> g = ld_grad<GT, VW>(p.g, e);
    Vec<VW> wl = ld_f32<VW>(p.w_loc, e);
    Vec<VW> pr = (first || sgd) ? wl : ld_f32<VW>(p.pre, e);
    Vec<VW> wg;
    if (pull) wg = ld_f32<VW>(p.w, e);
    Vec<VW> r;
    const GroupScalars<PT, VW> sc(p.s, p.tt, e);
#pragma unroll
    for (int l = 0; l < VW; ++l)
        r.v[l] = sgd ? local_sgd_elem(g.get(l), wl.v[l], sc.at(l)) : glu_elem(g.get(l), wl.v[l], pr.v[l], sc.at(l));
    if (first || refresh) st_f32<VW>(p.pre, e, wl);
    if (pull) {
        st_f32<VW>(p.w_dev, e, r);
        st_f32<VW>(p.w_loc, e, wg);
    } else {
        st_f32<VW>(p.w_loc, e, r);
    }
}

// One worker's pull when its device weights are its local weights (kMergedDev): pre_weight takes
// the old local weight where the iteration writes pre_weight, the local weight takes the global one.
template <int VW> __device__ __forceinline__ void glu_merged_pull_at(const GluParams &p, int64_t e)
{
    const bool writes_pre = (p.flags & (kFirst | kRefresh)) && !(p.flags & kLocalSgd);
    Vec<VW> wg = ld_f32<VW>(p.w, e);
    if (writes_pre) st_f32<VW>(p.pre, e, ld_f32<VW>(p.w_loc, e));
    st_f32<VW>(p.w_loc, e, wg);
}

// Pull iteration of a context whose device weights are its local weights (kMergedDev): the
// server update, pre_weight = old local weight where the iteration writes pre_weight (only with
// k = 1 does a pull coincide with that), then every local weight takes the new global weight.
// The local update itself is skipped: its result would be overwritten before anyone could read it.
template <int GT, int VW, int B, bool PT>
__device__ __forceinline__ void step_merged_pull_at(const StepParams &p, int64_t e)
{
    const bool sgd = p.flags & kLocalSgd;
    const bool writes_pre = (p.flags & (kFirst | kRefresh)) && !sgd;
    Vec<VW> w = ld_f32<VW>(p.w, e);
    Vec<VW> mom = ld_f32<VW>(p.mom, e);
    Vec<VW> sum;
    const int per = p.per_batch;
    for (int i0 = 0; i0 < p.K; i0 += per) {
        Grad<GT, VW> g[B];
#pragma unroll
        for (int b = 0; b < B; ++b)
            if (b < per && i0 + b < p.K) g[b] = ld_grad<GT, VW>(p.g[i0 + b], e);
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (b < per && i0 + b < p.K) {
#pragma unroll
                for (int l = 0; l < VW; ++l)
                    sum.v[l] = (i0 + b == 0) ? g[b].get(l) : __fadd_rn(sum.v[l], g[b].get(l));
            }
        }
    }
    const GroupScalars<PT, VW> sc(p.s, p.tt, e);
#pragma unroll
    for (int l = 0; l < VW; ++l) server_elem(sum.v[l], w.v[l], mom.v[l], sc.at(l));
    if (writes_pre) {
        const int copies = p.shared_pre ? 1 : p.K;
        for (int i = 0; i < copies; ++i) st_f32<VW>(p.pre[i], e, ld_f32<VW>(p.w_loc[i], e));
    }
    st_f32<VW>(p.mom, e, mom);
    st_f32<VW>(p.w, e, w);
    for (int i = 0; i < p.K; ++i) st_f32<VW>(p.w_loc[i], e, w);
}

template <int GT, int VW, int B, bool PT>
__device__ __forceinline__ void step_at(const StepParams &p, int64_t e)
{
    const bool sgd = p.flags & kLocalSgd;      // plain-SGD updater: pre_weight is not involved at all
    const bool first = (p.flags & kFirst) && !sgd, refresh = (p.flags & kRefresh) && !sgd, pull = p.flags & kPull;
    Vec<VW> w = ld_f32<VW>(p.w, e);
    Vec<VW> mom = ld_f32<VW>(p.mom, e);
    Vec<VW> sum;
    // A shared pre_weight is read once per element instead of once per worker, and written
    // once: on the iterations that write it every worker's local weight holds the same pulled
    // global weight, so worker 0's value is everyone's.
    const bool shared = p.shared_pre != 0;
    Vec<VW> pre_shared;
    if (shared && !first && !sgd) pre_shared = ld_f32<VW>(p.pre[0], e);
    GroupScalars<PT, VW> sc(p.s, p.tt, e);
    const int per = p.per_batch;
    for (int i0 = 0; i0 < p.K; i0 += per) {
        Grad<GT, VW> g[B];
        Vec<VW> wl[B], pr[B];
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (b < per && i0 + b < p.K) {
                g[b] = ld_grad<GT, VW>(p.g[i0 + b], e);
                wl[b] = ld_f32<VW>(p.w_loc[i0 + b], e);
                if (!first && !shared && !sgd) pr[b] = ld_f32<VW>(p.pre[i0 + b], e);
            }
        }
#pragma unroll
        for (int b = 0; b < B; ++b) {
            if (b < per && i0 + b < p.K) {
                const int i = i0 + b;
                Vec<VW> r;
#pragma unroll
                for (int l = 0; l < VW; ++l) {
                    const float gl = g[b].get(l);
                    sum.v[l] = (i == 0) ? gl : __fadd_rn(sum.v[l], gl);
                    const float pl = (first || sgd) ? wl[b].v[l] : shared ? pre_shared.v[l] : pr[b].v[l];
                    r.v[l] = sgd ? local_sgd_elem(gl, wl[b].v[l], sc.at(l)) : glu_elem(gl, wl[b].v[l], pl, sc.at(l));
                }
                if ((first || refresh) && (!shared || i == 0)) st_f32<VW>(p.pre[i], e, wl[b]);
                st_f32<VW>(pull ? p.w_dev[i] : p.w_loc[i], e, r);
            }
        }
    }
#pragma unroll
    for (int l = 0; l < VW; ++l) server_elem(sum.v[l], w.v[l], mom.v[l], sc.at(l));
    st_f32<VW>(p.mom, e, mom);
    st_f32<VW>(p.w, e, w);
    if (pull)
        for (int i = 0; i < p.K; ++i) st_f32<VW>(p.w_loc[i], e, w);
}

// ---------------------------------------------------------------------------
// Kernels: grid-stride over the n/VW vectors of the arena.  Arena lengths are
// multiples of 4; with VW > 4 the remaining groups of 4 elements are finished by
// one thread with the 128-bit body.
// ---------------------------------------------------------------------------
#define SSD_SWEEP(n, VW, BODY, TAIL)                                                      \
    do {                                                                                  \
        const int64_t nvec = (n) / (VW);                                                  \
        const int64_t stride = (int64_t)gridDim.x * blockDim.x;                           \
        for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < nvec; v += stride) { \
            const int64_t e = v * (VW);                                                   \
            BODY;                                                                         \
        }                                                                                 \
        if ((VW) > 4 && blockIdx.x == 0 && threadIdx.x == 0) {                            \
            for (int64_t e = nvec * (VW); e < (n); e += 4) {                              \
                TAIL;                                                                     \
            }                                                                             \
        }                                                                                 \
    } while (0)

// Threads per block each kernel is compiled for: vectors of 16 hold twice the registers.
constexpr int threads_bound(int VW) { return VW == 16 ? kMaxThreads / 2 : kMaxThreads; }

// PT: per-tensor scalars from the table instead of the uniform ones.
template <int GT, int VW, int B, bool PT>
__global__ void __launch_bounds__(threads_bound(VW)) sync_kernel(const __grid_constant__ SyncParams p)
{
    SSD_SWEEP(p.n, VW, (sync_at<GT, VW, B, PT>(p, e)), (sync_at<GT, 4, B, PT>(p, e)));
}

template <int GT, int VW, bool PT>
__global__ void __launch_bounds__(threads_bound(VW)) glu_kernel(const __grid_constant__ GluParams p)
{
    SSD_SWEEP(p.n, VW, (glu_at<GT, VW, PT>(p, e)), (glu_at<GT, 4, PT>(p, e)));
}

template <int GT, int VW, int B, bool PT>
__global__ void __launch_bounds__(threads_bound(VW)) step_kernel(const __grid_constant__ StepParams p)
{
    SSD_SWEEP(p.n, VW, (step_at<GT, VW, B, PT>(p, e)), (step_at<GT, 4, B, PT>(p, e)));
}

// The two pull forms of a context with merged device weights, as kernels of their own so that the
// kernels above keep their register budgets.
template <int GT, int VW, int B, bool PT>
__global__ void __launch_bounds__(threads_bound(VW)) step_merged_pull_kernel(const __grid_constant__ StepParams p)
{
    SSD_SWEEP(p.n, VW, (step_merged_pull_at<GT, VW, B, PT>(p, e)), (step_merged_pull_at<GT, 4, B, PT>(p, e)));
}

template <int VW>
__global__ void __launch_bounds__(threads_bound(VW)) glu_merged_pull_kernel(const __grid_constant__ GluParams p)
{
    SSD_SWEEP(p.n, VW, (glu_merged_pull_at<VW>(p, e)), (glu_merged_pull_at<4>(p, e)));
}

template <int VW> __device__ __forceinline__ void copy_at(const CopyParams &p, int64_t e)
{
    Vec<VW> x = ld_f32<VW>(p.src, e);
    for (int i = 0; i < p.K; ++i) st_f32<VW>(p.dst[i], e, x);
}

// dst[i] = src for K destinations (the pull of a freshly initialised or warm-up weight).
template <int VW>
__global__ void __launch_bounds__(threads_bound(VW)) copy_kernel(const __grid_constant__ CopyParams p)
{
    SSD_SWEEP(p.n, VW, (copy_at<VW>(p, e)), (copy_at<4>(p, e)));
}

}  // namespace ssd
