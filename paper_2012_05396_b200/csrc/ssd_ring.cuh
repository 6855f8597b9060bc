// The fused step with shared-memory staging: an alternative to step_kernel.
//
// One producer thread per block streams tile after tile of the inputs into a ring of
// shared-memory stages with 1-D bulk asynchronous copies (cp.async.bulk, the non-tensor
// form of TMA; no multicast, no clusters), each stage guarded by a pair of mbarriers;
// 256 consumer threads take the values from shared memory, do the arithmetic of
// step_at and store the results straight to global memory.  A stage holds one tile
// (kRingTile elements) of one worker's three inputs (gradient, local weight,
// pre_weight) or, as the last stage of a tile, of w and mom; the K-way sum lives in the
// consumers' registers across the K stages of a tile.  Bytes in flight are then set by
// the number of stages, not by registers and occupancy.
//
// Measured on B200 this is NOT faster than the register path (plain iterations about
// equal at best, write-heavy iterations 8 % slower), so it is off by default; it is kept,
// tested for bit-exactness, so that the comparison can be repeated
// (ssd_set_staging, `sweep --staging N`).
//
// Every wait on an mbarrier is bounded: a thread that runs out of tries records the
// fact in g_ring_error and leaves; no thread waits for ever.
#pragma once

#include "ssd_kernels.cuh"

namespace ssd {

constexpr int kRingTile = 2048;                    // elements per tile per stream
constexpr int kRingSlotBytes = kRingTile * 4;      // one float32 stream segment
constexpr int kRingStageBytes = 3 * kRingSlotBytes;
constexpr int kRingConsumers = 256;                // each owns 8 consecutive elements of a tile
constexpr int kRingThreads = kRingConsumers + 32;  // plus the producer's warp
constexpr int kRingWaitLimit = 1 << 20;
constexpr int kRingMaxStages = 8;

// Set to 1 by any thread whose bounded wait ran out (never happens in a correct run).
__device__ int g_ring_error;

__device__ __forceinline__ uint32_t ring_s32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t *b, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ring_s32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *b, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ring_s32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *b)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(ring_s32(b)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t *b, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok) : "r"(ring_s32(b)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *b, uint32_t parity)
{
    for (int it = 0; it < kRingWaitLimit; ++it)
        if (mbar_try(b, parity)) return true;
    atomicExch(&g_ring_error, 1);
    return false;
}
// Bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(ring_s32(dst)), "l"(src), "r"(bytes), "r"(ring_s32(bar)) : "memory");
}

__device__ __forceinline__ Vec<4> lds_f32x4(const float *p)
{
    const float4 t = *reinterpret_cast<const float4 *>(p);
    return Vec<4>{{t.x, t.y, t.z, t.w}};
}

// Four gradient values at element o of a staged gradient segment.
template <int GT> __device__ __forceinline__ Vec<4> lds_grad4(const float *slot, int o);
template <> __device__ __forceinline__ Vec<4> lds_grad4<kF32>(const float *slot, int o) { return lds_f32x4(slot + o); }
template <> __device__ __forceinline__ Vec<4> lds_grad4<kBF16>(const float *slot, int o)
{
    const uint2 t = *reinterpret_cast<const uint2 *>(reinterpret_cast<const uint16_t *>(slot) + o);
    return Vec<4>{{bf16_lo(t.x), bf16_hi(t.x), bf16_lo(t.y), bf16_hi(t.y)}};
}

// p: as for step_kernel (shared_pre == 0 and no kLocalSgd flag: the host keeps those on the
// register path); stages: 2..kRingMaxStages.  Dynamic shared memory: stages * kRingStageBytes
// + 2 * stages mbarriers.  p.n is a multiple of 4, every pointer 16-byte aligned.
template <int GT, bool PT>
__global__ void __launch_bounds__(kRingThreads) step_ring_kernel(const __grid_constant__ StepParams p, int stages)
{
    extern __shared__ __align__(128) unsigned char ring_smem[];
    float *stage_mem = reinterpret_cast<float *>(ring_smem);
    uint64_t *full = reinterpret_cast<uint64_t *>(ring_smem + static_cast<size_t>(stages) * kRingStageBytes);
    uint64_t *empty = full + stages;
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&full[s], 1);                      // the producer's expect_tx arrival
            mbar_init(&empty[s], kRingConsumers / 32);   // one arrival per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const bool first = p.flags & kFirst, refresh = p.flags & kRefresh, pull = p.flags & kPull;
    const int64_t ntiles = (p.n + kRingTile - 1) / kRingTile;
    constexpr uint32_t kGradBytesPerElem = GT == kBF16 ? 2 : 4;

    if (tid >= kRingConsumers) {
        if (tid != kRingConsumers) return;               // one producer thread
        uint32_t it = 0;
        for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
            const int64_t e0 = tile * kRingTile;
            const uint32_t cnt = static_cast<uint32_t>(p.n - e0 < kRingTile ? p.n - e0 : kRingTile);
            for (int i = 0; i <= p.K; ++i, ++it) {
                const int s = it % stages;
                const uint32_t phase = (it / stages) & 1;
                if (!mbar_wait(&empty[s], phase ^ 1)) return;      // consumers are done with this stage
                float *sb = stage_mem + static_cast<size_t>(s) * (kRingStageBytes / 4);
                if (i < p.K) {
                    mbar_expect_tx(&full[s], cnt * kGradBytesPerElem + cnt * 4 * (first ? 1 : 2));
                    bulk_g2s(sb, static_cast<const unsigned char *>(p.g[i]) + e0 * kGradBytesPerElem,
                             cnt * kGradBytesPerElem, &full[s]);
                    bulk_g2s(sb + kRingTile, p.w_loc[i] + e0, cnt * 4, &full[s]);
                    if (!first) bulk_g2s(sb + 2 * kRingTile, p.pre[i] + e0, cnt * 4, &full[s]);
                } else {
                    mbar_expect_tx(&full[s], cnt * 8);
                    bulk_g2s(sb, p.w + e0, cnt * 4, &full[s]);
                    bulk_g2s(sb + kRingTile, p.mom + e0, cnt * 4, &full[s]);
                }
            }
        }
        return;
    }

    uint32_t it = 0;
    const int le = tid * 8;                              // this thread's first element in a tile
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const int64_t e0 = tile * kRingTile;
        const int cnt = static_cast<int>(p.n - e0 < kRingTile ? p.n - e0 : kRingTile);
        const bool active[2] = {le < cnt, le + 4 < cnt};
        const GroupScalars<PT, 4> sc0(p.s, p.tt, e0 + le), sc1(p.s, p.tt, e0 + le + 4);
        Vec<4> sum[2];
        for (int i = 0; i < p.K; ++i, ++it) {
            const int s = it % stages;
            if (!mbar_wait(&full[s], (it / stages) & 1)) return;
            const float *sb = stage_mem + static_cast<size_t>(s) * (kRingStageBytes / 4);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (active[h]) {
                    const int o = le + 4 * h;
                    const Vec<4> g = lds_grad4<GT>(sb, o), wl = lds_f32x4(sb + kRingTile + o);
                    const Vec<4> pr = first ? wl : lds_f32x4(sb + 2 * kRingTile + o);
                    const Scalars &sc = h ? sc1.at(0) : sc0.at(0);
                    Vec<4> r;
#pragma unroll
                    for (int l = 0; l < 4; ++l) {
                        sum[h].v[l] = (i == 0) ? g.v[l] : __fadd_rn(sum[h].v[l], g.v[l]);
                        r.v[l] = glu_elem(g.v[l], wl.v[l], pr.v[l], sc);
                    }
                    if (first || refresh) st_f32<4>(p.pre[i], e0 + o, wl);
                    st_f32<4>(pull ? p.w_dev[i] : p.w_loc[i], e0 + o, r);
                }
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&empty[s]);
        }
        {
            const int s = it % stages;
            if (!mbar_wait(&full[s], (it / stages) & 1)) return;
            const float *sb = stage_mem + static_cast<size_t>(s) * (kRingStageBytes / 4);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (active[h]) {
                    const int o = le + 4 * h;
                    Vec<4> w = lds_f32x4(sb + o), mom = lds_f32x4(sb + kRingTile + o);
                    const Scalars &sc = h ? sc1.at(0) : sc0.at(0);
#pragma unroll
                    for (int l = 0; l < 4; ++l) server_elem(sum[h].v[l], w.v[l], mom.v[l], sc);
                    st_f32<4>(p.mom, e0 + o, mom);
                    st_f32<4>(p.w, e0 + o, w);
                    if (pull)
                        for (int i = 0; i < p.K; ++i) st_f32<4>(p.w_loc[i], e0 + o, w);
                }
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&empty[s]);
            ++it;
        }
    }
}

}  // namespace ssd
