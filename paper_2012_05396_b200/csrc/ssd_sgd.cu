// Host side of the SSD-SGD update library: context, argument validation, the
// schedule state machine of Algorithm 1 / Algorithm 2, and the kernel launches.
// The contract of every entry point is stated in include/ssd_sgd.h.
#include "ssd_sgd.h"
#include "ssd_kernels.cuh"
#include "ssd_ring.cuh"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <string>
#include <utility>
#include <vector>

namespace {

using namespace ssd;

constexpr int64_t kMaxArena = int64_t(1) << 40;
constexpr int64_t kL2ResidentBytes = 128 << 20;         // a step moving less than this stays within the 126 MB L2
constexpr int64_t kHostChunkElems = int64_t(1) << 24;   // ssd_step_host: default elements per pipelined chunk
constexpr int kMaxPreSlots = 8;                         // device slices of a host-resident pre_weight

struct Device {
    bool ready = false;
    int id = -1;
    int sms = 0;
};

// Byte range [lo, hi) of a buffer.
struct Range {
    uintptr_t lo, hi;
};

}  // namespace

struct ssd_ctx {
    std::vector<int64_t> offsets;     // element offset of each tensor
    int64_t n = 0;                    // arena length in elements
    ssd_hparams hp{};                 // resolved
    Scalars s{};
    float *w = nullptr, *mom = nullptr;
    float *w_loc[kMaxWorkers]{}, *pre[kMaxWorkers]{}, *w_dev[kMaxWorkers]{};
    bool has_workers = true;          // false: delay_k == 0 and no worker tables were given
    bool shared_pre = false;          // all K pre_weight pointers are the same buffer
    bool pre_on_device = true;        // false: created without pre_weight buffers (see ssd_set_host_pre_weight)
    bool merged_dev = false;          // w_dev[i] == w_loc[i] for every worker: no separate device weights
    // pre_weight kept in host memory: one pinned host arena, streamed through `pre_slots` device
    // slices of `host_chunk` elements by ssd_step_host
    float *host_pre = nullptr, *pre_slices = nullptr;
    int pre_slots = 0;
    int64_t host_chunk = kHostChunkElems;
    int64_t iter = 0, loc_update = 0;
    bool state32 = false;             // every state buffer is 32-byte aligned
    int threads = 0, blocks_per_sm = 0;     // 0: the kernel's default shape
    int force_vw = 0, force_batch = 0;      // 0: chosen from alignment and K
    int staging = 0;                        // > 0: fused step through a shared-memory ring of that many stages
    // per-tensor scalars: host copies of the multipliers and the caller's device table
    std::vector<float> lr_mult, wd_mult;
    void *tensor_table = nullptr;
    std::vector<unsigned char> table_image;   // what was last uploaded
    std::vector<unsigned char> static_image;  // the same for ssd_server_sync_update_static
    // ssd_step_host pipelines chunks over two side streams (copies in, copies out)
    cudaStream_t in_stream = nullptr, out_stream = nullptr;
    std::vector<cudaEvent_t> events;
    std::map<std::pair<const void *, int>, int> occupancy;   // (kernel, threads) -> blocks that fit per SM
    std::vector<Range> state_ranges;  // the state buffers' byte ranges, sorted by address, free of overlaps
    int64_t launches = 0;
    Device dev;
    std::string cuda_error;
};

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

float derive_sync_scale(float lr, float m, int32_t k)
{
    if (k <= 0) return 0.0f;
    return static_cast<float>((1.0 - static_cast<double>(m)) /
                              (static_cast<double>(lr) * static_cast<double>(k)));
}

ssd_status padded_total(const ssd_layout *layout, int64_t *total, std::vector<int64_t> *offsets)
{
    if (!layout || !layout->numel) return SSD_ERR_ARG;
    if (layout->num_tensors < 1) return SSD_ERR_LAYOUT;
    int64_t pos = 0;
    for (int32_t t = 0; t < layout->num_tensors; ++t) {
        const int64_t c = layout->numel[t];
        if (c < 0 || c >= kMaxArena) return SSD_ERR_LAYOUT;
        if (offsets) offsets->push_back(pos);
        pos += (c + 3) / 4 * 4;
        if (pos >= kMaxArena) return SSD_ERR_LAYOUT;
    }
    if (pos == 0) return SSD_ERR_LAYOUT;
    *total = pos;
    return SSD_OK;
}

void schedule_of(const ssd_ctx *c, int64_t n, int32_t *stage, int32_t *flags)
{
    const int64_t W = c->hp.warmup_iters, k = c->hp.delay_k;
    if (k == 0 || n < W) {
        *stage = SSD_STAGE_WARMUP;
        *flags = (k != 0 && n == W - 1) ? SSD_FLAG_COPY : 0;
        return;
    }
    const int64_t d = n - W;
    int32_t f = 0;
    if (d == 0) f |= SSD_FLAG_FIRST;
    if (d > 0 && d % k == 0) f |= SSD_FLAG_REFRESH;
    if (d % k == k - 1) f |= SSD_FLAG_PULL;
    *stage = SSD_STAGE_DELAY;
    *flags = f;
}

ssd_status cuda_fail(ssd_ctx *c, cudaError_t e)
{
    c->cuda_error = cudaGetErrorString(e);
    return SSD_ERR_CUDA;
}

ssd_status ensure_device(ssd_ctx *c)
{
    if (c->dev.ready) return SSD_OK;
    int id = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&id);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, id);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        return cuda_fail(c, e);
    }
    c->dev.id = id;
    c->dev.sms = sms;
    c->dev.ready = true;
    return SSD_OK;
}

// Launch shape of one sweep: elements per thread per trip, workers whose loads are issued
// together, threads per block, resident blocks per SM (0 = as many as fit).
struct Shape {
    int vw, batch, threads, per_sm;
};

// Grid for a sweep over n elements: at most `per_sm` resident blocks per SM, never more than
// fit, so that the grid is a single wave and every block's trips are equally long.
template <typename Kernel>
ssd_status grid_for(ssd_ctx *c, Kernel kernel, int64_t n, const Shape &sh, int *grid)
{
    // resident blocks per SM of this kernel at this block size: asked once, then remembered
    const std::pair<const void *, int> key(reinterpret_cast<const void *>(kernel), sh.threads);
    int fit = 0;
    auto hit = c->occupancy.find(key);
    if (hit != c->occupancy.end()) {
        fit = hit->second;
    } else {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, kernel, sh.threads, 0);
        if (e != cudaSuccess) return cuda_fail(c, e);
        if (fit < 1) fit = 1;
        c->occupancy[key] = fit;
    }
    const int per_sm = (sh.per_sm > 0 && sh.per_sm < fit) ? sh.per_sm : fit;
    const int64_t nvec = n / sh.vw;
    int64_t need = (nvec + sh.threads - 1) / sh.threads;
    if (need < 1) need = 1;
    const int64_t wave = static_cast<int64_t>(c->dev.sms) * per_sm;
    *grid = static_cast<int>(need < wave ? need : wave);
    return SSD_OK;
}

template <typename Kernel, typename Params>
ssd_status launch(ssd_ctx *c, Kernel kernel, const Params &p, int64_t n, const Shape &sh, cudaStream_t stream)
{
    ssd_status st = ensure_device(c);
    if (st != SSD_OK) return st;
    int grid = 1;
    st = grid_for(c, kernel, n, sh, &grid);
    if (st != SSD_OK) return st;
    kernel<<<grid, sh.threads, 0, stream>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return SSD_OK;
}

bool aligned32(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }

// Largest vector a launch may use.  8 elements per thread (256-bit accesses) need 32-byte aligned
// float32 buffers; bfloat16 gradients are then read 128 bits at a time, which every buffer allows.
// 16 elements per thread read bfloat16 gradients 256 bits at a time, so those need 32 bytes too.
// `lo` is the first element of a range launch: it shifts every buffer's alignment.
int max_vector(const ssd_ctx *c, bool state32, const void *const *grads, int count, int64_t lo,
               const void *extra = nullptr)
{
    if (!state32 || lo % 8 != 0 || (extra && !aligned32(extra))) return 4;
    bool grads32 = true;
    for (int i = 0; i < count; ++i) grads32 = grads32 && aligned32(grads[i]);
    if (c->hp.grad_dtype == SSD_F32) return grads32 ? 16 : 4;
    return (grads32 && lo % 16 == 0) ? 16 : 8;
}

// The caller's overrides (ssd_set_kernel_shape, ssd_set_launch) on top of a default shape.
Shape finish_shape(const ssd_ctx *c, Shape sh, int max_vw, int max_batch)
{
    if (c->force_vw) sh.vw = c->force_vw;
    if (sh.vw > max_vw) sh.vw = max_vw;
    if (c->force_batch) sh.batch = c->force_batch;
    if (sh.batch > max_batch) sh.batch = max_batch;
    if (c->threads) {
        sh.threads = c->threads;
        sh.per_sm = c->blocks_per_sm;
    } else if (c->blocks_per_sm) {
        sh.per_sm = c->blocks_per_sm;
    }
    if (sh.threads > threads_bound(sh.vw)) sh.threads = threads_bound(sh.vw);
    return sh;
}

// Default shapes.  These kernels are limited by how well HBM is kept busy, which depends on
// the bytes in flight per SM (threads x loads per thread x bytes per load) and on the mix of
// reads and writes: too few bytes in flight cannot cover the DRAM latency, too many lower
// the DRAM efficiency again, sooner so when a large share of the traffic is writes.  The
// values below are the measured optima on B200 (arenas of 25M..138M elements).
Shape sync_shape(const ssd_ctx *c, int max_vw, int flags = 0)
{
    const int K = c->hp.K;
    Shape sh;
    if (flags & kCopy) {
        // K + 2 stores per element behind the K + 2 loads (the hand-over iteration of the warm-up
        // stage, and every pull of a context with merged device weights): 44 % of the traffic is
        // writes, and 384 threads per SM is the optimum whatever K (6.5-6.65 TB/s float32,
        // 6.25-6.5 bfloat16, against 5.9-6.1 with the shapes below)
        // (with one to three float32 workers there are too few streams for that: vectors of 16, or 512
        // threads per SM for two workers, bring 5.2-6.2 TB/s to 6.4-6.6)
        const bool bf16 = c->hp.grad_dtype == SSD_BF16;
        Shape copy_shape = Shape{8, 4, 128, 3};
        if (max_vw >= 16 && (bf16 || K == 1 || K == 3)) copy_shape = Shape{16, 2, 128, 3};
        else if (!bf16 && K == 2) copy_shape = Shape{8, 2, 128, 4};
        return finish_shape(c, copy_shape, max_vw, 8);
    }
    // (the batch is an upper bound: the K workers go in ceil(K / batch) batches of equal size)
    if (c->hp.grad_dtype == SSD_BF16) {
        // bfloat16 gradients: vectors of 16 fetch them with 256-bit loads like the float32 state
        // (with vectors of 8 a warp asks for 512 contiguous bytes of a gradient stream at a time and
        // the kernel stays 7 % below its float32 twin)
        if (K >= 16) sh = Shape{16, 8, 128, 3};
        else if (K >= 7) sh = Shape{16, 8, 128, 4};
        else if (K >= 5) sh = Shape{16, 8, 128, 3};
        else if (K == 4) sh = Shape{16, 4, 128, 3};
        else if (K == 3) sh = Shape{8, 4, 128, 6};
        else if (K == 2) sh = Shape{16, 1, 128, 6};
        else sh = Shape{16, 1, 128, 4};
        if (max_vw < 16) sh = K >= 3 ? Shape{8, 4, 128, 6} : Shape{8, 1, 128, K == 1 ? 4 : 6};
    } else {
        if (K == 4) sh = Shape{8, 4, 256, 3};
        else if (K >= 8) sh = Shape{8, 4, 128, 5};
        else if (K >= 5) sh = Shape{8, 8, 128, 4};
        else if (K == 3) sh = Shape{16, 4, 128, 3};
        else if (K == 2) sh = Shape{16, 2, 128, 3};
        else sh = Shape{8, 1, 128, 6};
        if (max_vw < 16 && K < 4) sh = K == 3 ? Shape{8, 4, 128, 5} : Shape{8, 1, 128, 6};
    }
    return finish_shape(c, sh, max_vw, 8);
}

Shape step_shape(const ssd_ctx *c, int flags, bool shared_pre, int max_vw, int64_t count)
{
    // Iterations that add K stores per element (pull; refresh or first call with one pre_weight
    // per worker) are write-heavy: 512 threads per SM with vectors of 8.  The others: 640 threads
    // per SM.  Vectors of 16 (384 threads per SM) win where gradients are bfloat16 and the iteration
    // is write-heavy, and on plain iterations with one or two workers.
    const int K = c->hp.K;
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    const bool sgd = c->hp.local_updater == SSD_LOCAL_SGD;
    const bool k_extra_stores = (flags & kPull) || (!shared_pre && !sgd && (flags & (kRefresh | kFirst)));
    Shape sh = k_extra_stores ? Shape{8, 1, 128, 4} : Shape{8, 1, 128, 5};
    // plain iterations with many workers: two workers' loads per thread at 512 threads per SM (+1.4 %)
    if (!k_extra_stores && K >= 12) sh = Shape{8, 2, 128, 4};
    if (max_vw >= 16) {
        if (k_extra_stores && bf16) sh = Shape{16, 1, 128, 3};
        if (!k_extra_stores && (K == 1 || (K == 2 && !bf16))) sh = Shape{16, 1, 128, 3};
        if (!k_extra_stores && K == 4 && !bf16) sh = Shape{16, 2, 128, 3};
    }
    // One shared pre_weight (also a slice of a host-resident one): K fewer read streams, so two
    // workers' loads per thread keep as many bytes in flight; measured at 2^26 elements, K = 4..32:
    // plain and refresh iterations +2.5 % (float32, K >= 8) and +4..8 % (bfloat16, which sat at 5.9-6.3
    // TB/s before); pull iterations +2.7 % (float32) and +2..5 % (bfloat16, vectors of 8 again).
    if (shared_pre && !sgd && K >= 4) {
        if (!(flags & kPull)) {
            if (bf16 || K >= 8) sh = Shape{8, 2, 128, 5};
        } else if (bf16) {
            sh = Shape{8, 1, 128, 5};
        } else {
            sh = K >= 8 ? Shape{8, 2, 128, 3} : Shape{16, 1, 128, 3};
        }
    }
    // Plain-SGD local updater: no pre_weight streams either.  Pull iterations are half writes: 384
    // threads per SM with two workers' loads per thread (float32, +2.3 %), vectors of 8 at 640 threads
    // per SM (bfloat16: 6.3-6.4 TB/s against 5.7-5.9 with the vectors of 16 of the GLU form); the other
    // iterations with bfloat16 gradients and few workers want two workers' loads per thread (+5 %).
    if (sgd && K >= 4) {
        if (flags & kPull) sh = bf16 ? Shape{8, 1, 128, 5} : Shape{8, 2, 128, 3};
        else if (bf16 && K < 12) sh = Shape{8, 2, 128, 5};
    }
    // A step whose whole traffic fits in L2 (ResNet-20/56 sized arenas) is bound by latency, not by
    // DRAM: smaller vectors spread it over more threads, and two workers' loads per thread halve the
    // number of dependent round trips.
    const int64_t sg = bf16 ? 2 : 4;
    if (count * (K * (sg + 12) + 16) < kL2ResidentBytes) sh = Shape{4, 2, 64, 0};
    sh = finish_shape(c, sh, max_vw, 4);
    // batches that would spill registers under the kernels' thread bounds
    if (sh.vw >= 8 && sh.batch > 2) sh.batch = 2;
    return sh;
}

Shape glu_shape(const ssd_ctx *c, int max_vw)
{
    Shape sh = max_vw >= 16 ? Shape{16, 1, 128, 0} : Shape{8, 1, 256, 0};
    // bfloat16 gradients on long arenas: 640 threads per SM instead of all that fit (768)
    if (max_vw >= 16 && c->hp.grad_dtype == SSD_BF16 && c->n >= (int64_t(1) << 26)) sh.per_sm = 5;
    return finish_shape(c, sh, max_vw, 1);
}

size_t table_end_bytes(const ssd_ctx *c) { return (c->offsets.size() * sizeof(int64_t) + 15) / 16 * 16; }
size_t table_bytes(const ssd_ctx *c) { return table_end_bytes(c) + c->offsets.size() * sizeof(float4); }

TensorTable table_of(const ssd_ctx *c)
{
    TensorTable tt{};
    if (c->tensor_table) {
        tt.end = static_cast<const int64_t *>(c->tensor_table);
        tt.scal = reinterpret_cast<const float4 *>(static_cast<const unsigned char *>(c->tensor_table) +
                                                   table_end_bytes(c));
        tt.T = static_cast<int>(c->offsets.size());
    }
    return tt;
}

// The per-tensor table as the kernels read it: T tensor ends (int64, padded to 16 bytes), then T
// float4 {lr, wd, lr_local, c}.  Tensor t: lr*lr_mult[t], wd*wd_mult[t], lr_local*lr_mult[t] (one
// float multiplication each) and the grad_sync scale of its own lr.  NULL multipliers are all 1.
void build_table_image(const ssd_ctx *c, const float *lr_mult, const float *wd_mult,
                       std::vector<unsigned char> *image)
{
    const size_t T = c->offsets.size();
    image->assign(table_bytes(c), 0);
    int64_t *end = reinterpret_cast<int64_t *>(image->data());
    float4 *scal = reinterpret_cast<float4 *>(image->data() + table_end_bytes(c));
    for (size_t t = 0; t < T; ++t) {
        end[t] = t + 1 < T ? c->offsets[t + 1] : c->n;
        const float lm = lr_mult ? lr_mult[t] : 1.0f, wm = wd_mult ? wd_mult[t] : 1.0f;
        const float lr_t = c->hp.lr * lm;
        const float wd_t = c->hp.wd * wm;
        const float lr_loc_t = c->hp.lr_local * lm;
        scal[t] = make_float4(lr_t, wd_t, lr_loc_t, derive_sync_scale(lr_t, c->hp.momentum, c->hp.delay_k));
    }
}

// Rebuilds the context's table from its current hyper-parameters and multipliers and enqueues
// the upload into the caller's device table.
ssd_status upload_table(ssd_ctx *c, cudaStream_t stream)
{
    build_table_image(c, c->lr_mult.data(), c->wd_mult.data(), &c->table_image);
    ssd_status st = ensure_device(c);
    if (st != SSD_OK) return st;
    // the image is pageable host memory: the call returns once it has been staged
    cudaError_t e = cudaMemcpyAsync(c->tensor_table, c->table_image.data(), c->table_image.size(),
                                    cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(c, e);
    return SSD_OK;
}

bool ranges_overlap(const std::vector<Range> &r)      // r sorted by lo
{
    for (size_t x = 1; x < r.size(); ++x)
        if (r[x].lo < r[x - 1].hi) return true;
    return false;
}

// A gradient buffer is read-only input: it may not intersect any state buffer (a thread would
// read what another has already overwritten).  state_ranges is sorted and free of overlaps.
bool touches_state(const ssd_ctx *c, const void *g, size_t bytes)
{
    const uintptr_t lo = reinterpret_cast<uintptr_t>(g), hi = lo + bytes;
    auto it = std::upper_bound(c->state_ranges.begin(), c->state_ranges.end(), lo,
                               [](uintptr_t v, const Range &r) { return v < r.hi; });   // first range ending after lo
    return it != c->state_ranges.end() && it->lo < hi;
}

size_t grad_bytes(const ssd_ctx *c) { return static_cast<size_t>(c->n) * (c->hp.grad_dtype == SSD_BF16 ? 2 : 4); }

// The GLU rule needs pre_weight; a context created without pre_weight buffers can run its delay
// stage only through ssd_step_host with a host-resident pre_weight.
bool lacks_device_pre(const ssd_ctx *c) { return c->hp.local_updater == SSD_LOCAL_GLU && !c->pre_on_device; }

// Elements of one device slice of a host-resident pre_weight: a chunk, or the whole arena if shorter.
int64_t slice_elems(const ssd_ctx *c) { return c->host_chunk < c->n ? c->host_chunk : c->n; }

ssd_status check_grads(const ssd_ctx *c, const void *const *grads)
{
    if (!grads) return SSD_ERR_ARG;
    const size_t bytes = grad_bytes(c);
    for (int i = 0; i < c->hp.K; ++i) {
        if (!grads[i]) return SSD_ERR_ARG;
        if (!aligned16(grads[i])) return SSD_ERR_ALIGN;
        if (touches_state(c, grads[i], bytes)) return SSD_ERR_ARG;
    }
    return SSD_OK;
}

// K workers in ceil(K / batch) batches of equal size (the last one may be smaller by less than a batch).
int even_batch(int K, int batch)
{
    const int batches = (K + batch - 1) / batch;
    return (K + batches - 1) / batches;
}

template <int GT, int VW, bool PT>
ssd_status launch_sync_b(ssd_ctx *c, SyncParams &p, const Shape &sh, cudaStream_t stream)
{
    // eight float32 vectors of 16 in flight would spill: four is the most there
    constexpr int kMost = (VW == 16 && GT == kF32) ? 4 : 8;
    const int batch = sh.batch < kMost ? sh.batch : kMost;
    p.per_batch = even_batch(p.K, batch);
    switch (batch) {
    case 1: return launch(c, sync_kernel<GT, VW, 1, PT>, p, p.n, sh, stream);
    case 2: return launch(c, sync_kernel<GT, VW, 2, PT>, p, p.n, sh, stream);
    case 4: return launch(c, sync_kernel<GT, VW, 4, PT>, p, p.n, sh, stream);
    default: return launch(c, sync_kernel<GT, VW, kMost, PT>, p, p.n, sh, stream);
    }
}

template <bool PT>
ssd_status launch_sync_t(ssd_ctx *c, SyncParams &p, const Shape &sh, cudaStream_t stream)
{
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    if (sh.vw == 16)
        return bf16 ? launch_sync_b<kBF16, 16, PT>(c, p, sh, stream) : launch_sync_b<kF32, 16, PT>(c, p, sh, stream);
    if (sh.vw == 8)
        return bf16 ? launch_sync_b<kBF16, 8, PT>(c, p, sh, stream) : launch_sync_b<kF32, 8, PT>(c, p, sh, stream);
    return bf16 ? launch_sync_b<kBF16, 4, PT>(c, p, sh, stream) : launch_sync_b<kF32, 4, PT>(c, p, sh, stream);
}

// Gradient pointer advanced by `lo` elements of the context's gradient type.
const void *grad_at(const ssd_ctx *c, const void *g, int64_t lo)
{
    return static_cast<const unsigned char *>(g) + lo * (c->hp.grad_dtype == SSD_BF16 ? 2 : 4);
}

// The launch functions take an element range [lo, lo + count) of the arena (lo a multiple of 4, as
// tensor offsets are; max_vector narrows the accesses where lo shifts a buffer's alignment);
// count < 0 means the whole arena.
ssd_status launch_sync(ssd_ctx *c, const void *const *grads, int flags, cudaStream_t stream,
                       int64_t lo = 0, int64_t count = -1)
{
    SyncParams p{};
    for (int i = 0; i < c->hp.K; ++i) {
        p.g[i] = grad_at(c, grads[i], lo);
        p.w_loc[i] = c->w_loc[i] ? c->w_loc[i] + lo : nullptr;
    }
    p.w = c->w + lo;
    p.mom = c->mom + lo;
    p.n = count < 0 ? c->n : count;
    p.K = c->hp.K;
    p.flags = flags;
    p.s = c->s;
    const bool state32 = (flags & kCopy) ? c->state32 : (aligned32(c->w) && aligned32(c->mom));
    p.tt = table_of(c);
    p.tt.base = lo;
    const Shape sh = sync_shape(c, max_vector(c, state32, grads, c->hp.K, lo), flags);
    return p.tt.T ? launch_sync_t<true>(c, p, sh, stream) : launch_sync_t<false>(c, p, sh, stream);
}

template <bool PT>
ssd_status launch_glu_t(ssd_ctx *c, const GluParams &p, const Shape &sh, cudaStream_t stream)
{
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    if (sh.vw == 16)
        return bf16 ? launch(c, glu_kernel<kBF16, 16, PT>, p, p.n, sh, stream)
                    : launch(c, glu_kernel<kF32, 16, PT>, p, p.n, sh, stream);
    if (sh.vw == 8)
        return bf16 ? launch(c, glu_kernel<kBF16, 8, PT>, p, p.n, sh, stream)
                    : launch(c, glu_kernel<kF32, 8, PT>, p, p.n, sh, stream);
    return bf16 ? launch(c, glu_kernel<kBF16, 4, PT>, p, p.n, sh, stream)
                : launch(c, glu_kernel<kF32, 4, PT>, p, p.n, sh, stream);
}

ssd_status launch_glu(ssd_ctx *c, int worker, const void *grad, int flags, cudaStream_t stream)
{
    GluParams p{};
    p.g = grad;
    p.w_loc = c->w_loc[worker];
    p.pre = c->pre[worker];                    // NULL only with the plain-SGD updater, which never touches it
    p.w_dev = c->w_dev[worker];
    p.w = c->w;
    p.n = c->n;
    p.flags = flags | (c->hp.local_updater == SSD_LOCAL_SGD ? kLocalSgd : 0);
    p.s = c->s;
    p.tt = table_of(c);
    if (c->merged_dev && (flags & kPull)) {
        // no separate device weights: the pull is all that is left of this worker's iteration
        p.flags |= kMergedDev;
        const Shape sh = finish_shape(c, Shape{8, 1, 256, 0}, c->state32 ? 8 : 4, 1);
        if (sh.vw == 8) return launch(c, glu_merged_pull_kernel<8>, p, p.n, sh, stream);
        return launch(c, glu_merged_pull_kernel<4>, p, p.n, sh, stream);
    }
    const Shape sh = glu_shape(c, max_vector(c, c->state32, &grad, 1, 0));
    return p.tt.T ? launch_glu_t<true>(c, p, sh, stream) : launch_glu_t<false>(c, p, sh, stream);
}

template <int GT, int VW, bool PT>
ssd_status launch_step_b(ssd_ctx *c, StepParams &p, const Shape &sh, cudaStream_t stream)
{
    // step_shape keeps the batch at 2 or below for vectors of 8 and 16 (4 would spill)
    constexpr int kMost = VW == 4 ? 4 : 2;
    const int batch = sh.batch < kMost ? sh.batch : kMost;
    p.per_batch = even_batch(p.K, batch);
    switch (batch) {
    case 1: return launch(c, step_kernel<GT, VW, 1, PT>, p, p.n, sh, stream);
    case 2: return launch(c, step_kernel<GT, VW, 2, PT>, p, p.n, sh, stream);
    default: return launch(c, step_kernel<GT, VW, kMost, PT>, p, p.n, sh, stream);
    }
}

template <bool PT>
ssd_status launch_step_t(ssd_ctx *c, StepParams &p, const Shape &sh, cudaStream_t stream)
{
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    if (sh.vw == 16)
        return bf16 ? launch_step_b<kBF16, 16, PT>(c, p, sh, stream) : launch_step_b<kF32, 16, PT>(c, p, sh, stream);
    if (sh.vw == 8)
        return bf16 ? launch_step_b<kBF16, 8, PT>(c, p, sh, stream) : launch_step_b<kF32, 8, PT>(c, p, sh, stream);
    return bf16 ? launch_step_b<kBF16, 4, PT>(c, p, sh, stream) : launch_step_b<kF32, 4, PT>(c, p, sh, stream);
}

// Pull iteration that also writes pre_weight (k = 1) of a context with merged device weights.  Its
// gradient loads are batched like the server kernel's (the same limits on loads in flight).
template <int GT, int VW, bool PT>
ssd_status launch_merged_pull_b(ssd_ctx *c, StepParams &p, const Shape &sh, cudaStream_t stream)
{
    constexpr int kMost = (VW == 16 && GT == kF32) ? 4 : 8;
    const int batch = sh.batch < kMost ? sh.batch : kMost;
    p.per_batch = even_batch(p.K, batch);
    switch (batch) {
    case 1: return launch(c, step_merged_pull_kernel<GT, VW, 1, PT>, p, p.n, sh, stream);
    case 2: return launch(c, step_merged_pull_kernel<GT, VW, 2, PT>, p, p.n, sh, stream);
    case 4: return launch(c, step_merged_pull_kernel<GT, VW, 4, PT>, p, p.n, sh, stream);
    default: return launch(c, step_merged_pull_kernel<GT, VW, kMost, PT>, p, p.n, sh, stream);
    }
}

template <bool PT>
ssd_status launch_merged_pull_t(ssd_ctx *c, StepParams &p, const Shape &sh, cudaStream_t stream)
{
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    if (sh.vw == 16)
        return bf16 ? launch_merged_pull_b<kBF16, 16, PT>(c, p, sh, stream) : launch_merged_pull_b<kF32, 16, PT>(c, p, sh, stream);
    if (sh.vw == 8)
        return bf16 ? launch_merged_pull_b<kBF16, 8, PT>(c, p, sh, stream) : launch_merged_pull_b<kF32, 8, PT>(c, p, sh, stream);
    return bf16 ? launch_merged_pull_b<kBF16, 4, PT>(c, p, sh, stream) : launch_merged_pull_b<kF32, 4, PT>(c, p, sh, stream);
}

// The shared-memory ring covers the common case; the rest stays on the register path.  Its bulk
// copies need 16-byte aligned sources and sizes, which bfloat16 gradients give only for ranges that
// start and end on multiples of 8 elements.
bool ring_can_run(const ssd_ctx *c, bool shared_pre, int64_t lo, int64_t count)
{
    if (shared_pre || c->hp.local_updater != SSD_LOCAL_GLU) return false;
    if (c->hp.grad_dtype == SSD_BF16 && (lo % 8 != 0 || count % 8 != 0)) return false;
    return true;
}

template <typename Kernel>
ssd_status launch_ring(ssd_ctx *c, Kernel kernel, const StepParams &p, cudaStream_t stream)
{
    ssd_status st = ensure_device(c);
    if (st != SSD_OK) return st;
    const int stages = c->staging;
    const size_t smem = static_cast<size_t>(stages) * kRingStageBytes + 2 * stages * sizeof(uint64_t);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(c, e);
    const int64_t ntiles = (p.n + kRingTile - 1) / kRingTile;
    const int grid = static_cast<int>(ntiles < c->dev.sms ? ntiles : c->dev.sms);    // one block per SM
    kernel<<<grid, kRingThreads, smem, stream>>>(p, stages);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(c, e);
    c->launches += 1;
    return SSD_OK;
}

ssd_status launch_step_ring(ssd_ctx *c, const StepParams &p, cudaStream_t stream)
{
    const bool bf16 = c->hp.grad_dtype == SSD_BF16;
    if (p.tt.T)
        return bf16 ? launch_ring(c, step_ring_kernel<kBF16, true>, p, stream)
                    : launch_ring(c, step_ring_kernel<kF32, true>, p, stream);
    return bf16 ? launch_ring(c, step_ring_kernel<kBF16, false>, p, stream)
                : launch_ring(c, step_ring_kernel<kF32, false>, p, stream);
}

// pre_slice: when not NULL, the one pre_weight of all workers for exactly this range, at
// pre_slice[0 .. count) (a device slice of a host-resident pre_weight); the context's own
// pre_weight pointers are then not used.
ssd_status launch_step(ssd_ctx *c, const void *const *grads, int flags, cudaStream_t stream,
                       int64_t lo = 0, int64_t count = -1, float *pre_slice = nullptr)
{
    const bool writes_pre = (flags & (kFirst | kRefresh)) && c->hp.local_updater == SSD_LOCAL_GLU;
    // Merged device weights, pull iteration: the local update's result would be overwritten at once,
    // so what remains is the server update and K stores of the new global weight, which is the
    // server kernel's hand-over form ...
    if (c->merged_dev && (flags & kPull) && !writes_pre) return launch_sync(c, grads, kCopy, stream, lo, count);
    StepParams p{};
    const bool shared = c->shared_pre || pre_slice;
    for (int i = 0; i < c->hp.K; ++i) {
        p.g[i] = grad_at(c, grads[i], lo);
        p.w_loc[i] = c->w_loc[i] + lo;
        p.pre[i] = pre_slice ? pre_slice : c->pre[i] ? c->pre[i] + lo : nullptr;
        p.w_dev[i] = c->w_dev[i] + lo;
    }
    p.w = c->w + lo;
    p.mom = c->mom + lo;
    p.n = count < 0 ? c->n : count;
    p.K = c->hp.K;
    p.flags = flags | (c->hp.local_updater == SSD_LOCAL_SGD ? kLocalSgd : 0);
    p.shared_pre = shared ? 1 : 0;
    p.s = c->s;
    p.tt = table_of(c);
    p.tt.base = lo;
    if (c->merged_dev && (flags & kPull)) {
        // ... and with k = 1, where every pull also writes pre_weight, a kernel of its own
        p.flags |= kMergedDev;
        // K more loads than the hand-over form (the old local weights): vectors of 16, more loads per batch
        // (6.5-6.6 TB/s at 2^26 elements against 5.7 float32 / 6.25 bfloat16 with the hand-over shape)
        const int max_vw = max_vector(c, c->state32, grads, c->hp.K, lo, pre_slice);
        const Shape wide = c->hp.grad_dtype == SSD_BF16 ? Shape{16, 8, 128, 3} : Shape{16, 4, 128, 4};
        const Shape sh = max_vw >= 16 ? finish_shape(c, wide, max_vw, 8) : sync_shape(c, max_vw, kCopy);
        return p.tt.T ? launch_merged_pull_t<true>(c, p, sh, stream) : launch_merged_pull_t<false>(c, p, sh, stream);
    }
    if (c->staging && ring_can_run(c, shared, lo, p.n)) return launch_step_ring(c, p, stream);
    const Shape sh = step_shape(c, flags, shared, max_vector(c, c->state32, grads, c->hp.K, lo, pre_slice), p.n);
    return p.tt.T ? launch_step_t<true>(c, p, sh, stream) : launch_step_t<false>(c, p, sh, stream);
}

ssd_status launch_copy(ssd_ctx *c, int first_worker, int count, cudaStream_t stream)
{
    CopyParams p{};
    for (int i = 0; i < count; ++i) p.dst[i] = c->w_loc[first_worker + i];
    p.src = c->w;
    p.n = c->n;
    p.K = count;
    Shape sh = finish_shape(c, Shape{8, 1, 256, 0}, c->state32 ? 8 : 4, 1);
    if (sh.vw == 8) return launch(c, copy_kernel<8>, p, p.n, sh, stream);
    return launch(c, copy_kernel<4>, p, p.n, sh, stream);
}

void advance(ssd_ctx *c)
{
    int32_t stage, flags;
    schedule_of(c, c->iter, &stage, &flags);
    c->iter += 1;
    if (stage == SSD_STAGE_DELAY) c->loc_update += 1;
}

// ---------------------------------------------------------------------------
// Per-tensor table in static device memory, for ssd_server_sync_update_static.
// Same layout as the caller-allocated table (T tensor ends padded to 16 bytes, then T
// float4 {lr, wd, lr_local, c}), sized for SSD_STATIC_TABLE_MAX_TENSORS tensors.
// Every GPU that loads this library holds the 24 KB until the process exits.  In
// host code the name below is only a handle for cudaGetSymbolAddress; kernels get
// the device address that call returns.
// ---------------------------------------------------------------------------
constexpr size_t kStaticTableBytes = SSD_STATIC_TABLE_MAX_TENSORS * (sizeof(int64_t) + sizeof(float4));
static __device__ __align__(256) unsigned char g_static_tensor_table[kStaticTableBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_table_addr[kMaxDevices] = {};

// Device address of the static table on the current device (looked up once per device).
ssd_status static_table_address(ssd_ctx *c, unsigned char **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(c, e);
    if (dev < 0 || dev >= kMaxDevices) return SSD_ERR_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_table_addr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_tensor_table);
        if (e != cudaSuccess) return cuda_fail(c, e);
        g_static_table_addr[dev] = ptr;
    }
    *out = static_cast<unsigned char *>(g_static_table_addr[dev]);
    return SSD_OK;
}

}  // namespace

extern "C" {

ssd_status ssd_arena_numel(const ssd_layout *layout, int64_t *padded_numel)
{
    if (!padded_numel) return SSD_ERR_ARG;
    return padded_total(layout, padded_numel, nullptr);
}

ssd_status ssd_init(ssd_ctx **out, const ssd_layout *layout, const ssd_hparams *hp,
                    const ssd_buffers *b)
{
    if (!out) return SSD_ERR_ARG;
    *out = nullptr;
    if (!layout || !hp || !b) return SSD_ERR_ARG;
    if (hp->K < 1 || hp->K > SSD_MAX_WORKERS) return SSD_ERR_ARG;
    if (!(hp->lr > 0.0f) || !std::isfinite(hp->lr)) return SSD_ERR_ARG;
    if (!(hp->momentum >= 0.0f && hp->momentum < 1.0f)) return SSD_ERR_ARG;
    if (!std::isfinite(hp->wd)) return SSD_ERR_ARG;
    if (hp->warmup_iters < 0 || hp->delay_k < 0) return SSD_ERR_ARG;
    if (hp->grad_dtype != SSD_F32 && hp->grad_dtype != SSD_BF16) return SSD_ERR_ARG;
    if (hp->local_updater != SSD_LOCAL_GLU && hp->local_updater != SSD_LOCAL_SGD) return SSD_ERR_ARG;
    if (std::isinf(hp->lr_local) || std::isinf(hp->alpha) || std::isinf(hp->beta) ||
        std::isinf(hp->rescale))
        return SSD_ERR_ARG;
    // Without a delay stage (delay_k == 0) no worker state is ever touched: the tables may be NULL.
    // A NULL `pre` table with worker state means that pre_weight does not live in device memory
    // (ssd_set_host_pre_weight), or is never used (plain-SGD local updater).
    const bool workers = b->w_loc && b->w_dev && (hp->delay_k > 0 || b->pre);
    const bool device_pre = workers && b->pre;
    if (!b->w || !b->mom) return SSD_ERR_ARG;
    if (hp->delay_k > 0 && (!b->w_loc || !b->w_dev)) return SSD_ERR_ARG;

    ssd_ctx *c = new (std::nothrow) ssd_ctx;
    if (!c) return SSD_ERR_NOMEM;
    ssd_status st = padded_total(layout, &c->n, &c->offsets);
    if (st != SSD_OK) {
        delete c;
        return st;
    }
    // All K pre_weight pointers equal: one shared pre_weight (its K copies always hold the same
    // values, every worker takes it from the same pulled global weight).
    bool shared_pre = device_pre && hp->K > 1 && b->pre[0] != nullptr;
    for (int i = 1; shared_pre && i < hp->K; ++i) shared_pre = b->pre[i] == b->pre[0];
    // w_dev[i] == w_loc[i] for every worker: the device weights are the local weights themselves.
    // It has to hold for all workers or for none.
    int merged = 0;
    for (int i = 0; workers && i < hp->K; ++i) merged += (b->w_dev[i] && b->w_dev[i] == b->w_loc[i]) ? 1 : 0;
    const bool merged_dev = workers && merged == hp->K;
    if (merged != 0 && !merged_dev) st = SSD_ERR_ARG;
    std::vector<const void *> all{b->w, b->mom};
    for (int i = 0; workers && i < hp->K; ++i) {
        all.push_back(b->w_loc[i]);
        if (device_pre && (!shared_pre || i == 0)) all.push_back(b->pre[i]);
        if (!merged_dev) all.push_back(b->w_dev[i]);
    }
    for (const void *p : all) {
        if (!p) st = SSD_ERR_ARG;
        else if (!aligned16(p) && st == SSD_OK) st = SSD_ERR_ALIGN;
    }
    // No two state buffers may overlap: every element is read and written by one thread only,
    // which holds only if the buffers are disjoint.
    const size_t arena_bytes = static_cast<size_t>(c->n) * sizeof(float);
    for (const void *p : all) {
        const uintptr_t lo = reinterpret_cast<uintptr_t>(p);
        c->state_ranges.push_back(Range{lo, lo + arena_bytes});
    }
    std::sort(c->state_ranges.begin(), c->state_ranges.end(), [](const Range &x, const Range &y) { return x.lo < y.lo; });
    if (st == SSD_OK && ranges_overlap(c->state_ranges)) st = SSD_ERR_ARG;
    if (st != SSD_OK) {
        delete c;
        return st;
    }

    c->hp = *hp;
    if (std::isnan(hp->lr_local)) c->hp.lr_local = 4.0f * hp->lr;
    if (std::isnan(hp->alpha)) c->hp.alpha = 2.0f;
    if (std::isnan(hp->beta)) c->hp.beta = 0.5f;
    if (std::isnan(hp->rescale)) c->hp.rescale = static_cast<float>(1.0 / static_cast<double>(hp->K));
    c->s.lr = c->hp.lr;
    c->s.m = c->hp.momentum;
    c->s.wd = c->hp.wd;
    c->s.rescale = c->hp.rescale;
    c->s.lr_loc = c->hp.lr_local;
    c->s.alpha = c->hp.alpha;
    c->s.beta = c->hp.beta;
    c->s.c = derive_sync_scale(c->hp.lr, c->hp.momentum, c->hp.delay_k);
    c->w = b->w;
    c->mom = b->mom;
    c->has_workers = workers;
    c->shared_pre = shared_pre;
    c->pre_on_device = device_pre;
    c->merged_dev = merged_dev;
    c->state32 = true;
    for (const void *p : all) c->state32 = c->state32 && aligned32(p);
    for (int i = 0; workers && i < hp->K; ++i) {
        c->w_loc[i] = b->w_loc[i];
        c->pre[i] = device_pre ? b->pre[i] : nullptr;
        c->w_dev[i] = b->w_dev[i];
    }
    *out = c;
    return SSD_OK;
}

void ssd_destroy(ssd_ctx *ctx)
{
    if (!ctx) return;
    for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
    if (ctx->in_stream) cudaStreamDestroy(ctx->in_stream);
    if (ctx->out_stream) cudaStreamDestroy(ctx->out_stream);
    delete ctx;
}

ssd_status ssd_tensor_offset(const ssd_ctx *ctx, int32_t tensor, int64_t *elem_offset)
{
    if (!ctx || !elem_offset) return SSD_ERR_ARG;
    if (tensor < 0 || tensor >= static_cast<int32_t>(ctx->offsets.size())) return SSD_ERR_ARG;
    *elem_offset = ctx->offsets[tensor];
    return SSD_OK;
}

ssd_status ssd_schedule(const ssd_ctx *ctx, int64_t iter, int32_t *stage, int32_t *flags)
{
    if (!ctx || !stage || !flags || iter < 0) return SSD_ERR_ARG;
    schedule_of(ctx, iter, stage, flags);
    return SSD_OK;
}

ssd_status ssd_server_sync_update(ssd_ctx *ctx, const void *const *grads, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    ssd_status st = check_grads(ctx, grads);
    if (st != SSD_OK) return st;
    return launch_sync(ctx, grads, 0, static_cast<cudaStream_t>(cuda_stream));
}

ssd_status ssd_server_sync_update_static(ssd_ctx *ctx, const void *const *grads, const float *lr_mult,
                                         const float *wd_mult, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    ssd_status st = check_grads(ctx, grads);
    if (st != SSD_OK) return st;
    const size_t T = ctx->offsets.size();
    if (T > SSD_STATIC_TABLE_MAX_TENSORS) return SSD_ERR_TOO_LARGE;
    for (size_t t = 0; t < T; ++t) {
        if (lr_mult && (!(lr_mult[t] > 0.0f) || !std::isfinite(lr_mult[t]))) return SSD_ERR_ARG;
        if (wd_mult && !std::isfinite(wd_mult[t])) return SSD_ERR_ARG;
    }
    st = ensure_device(ctx);
    if (st != SSD_OK) return st;
    // the array's address differs per device: the context's device must be the current one
    int current = -1;
    cudaError_t e = cudaGetDevice(&current);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (current != ctx->dev.id) return SSD_ERR_STATE;
    unsigned char *table = nullptr;
    st = static_table_address(ctx, &table);
    if (st != SSD_OK) return st;

    // The image ssd_set_tensor_scales would upload, built by the same code and kept in the
    // context until the next call replaces it, written over the front of the static array
    // (bytes beyond it keep older contents and are never read).
    build_table_image(ctx, lr_mult, wd_mult, &ctx->static_image);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // pageable source: the call returns once the bytes have been staged
    e = cudaMemcpyAsync(table, ctx->static_image.data(), ctx->static_image.size(), cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e);

    SyncParams p{};
    for (int i = 0; i < ctx->hp.K; ++i) p.g[i] = grads[i];
    p.w = ctx->w;
    p.mom = ctx->mom;
    p.n = ctx->n;
    p.K = ctx->hp.K;
    p.flags = 0;
    p.s = ctx->s;
    p.tt.end = reinterpret_cast<const int64_t *>(table);
    p.tt.scal = reinterpret_cast<const float4 *>(table + table_end_bytes(ctx));
    p.tt.T = static_cast<int>(T);
    const bool state32 = aligned32(ctx->w) && aligned32(ctx->mom);
    const Shape sh = sync_shape(ctx, max_vector(ctx, state32, grads, ctx->hp.K, 0));
    return launch_sync_t<true>(ctx, p, sh, stream);
}

ssd_status ssd_worker_glu_update(ssd_ctx *ctx, int32_t worker, const void *grad, int32_t flags,
                                 void *cuda_stream)
{
    if (!ctx || !grad) return SSD_ERR_ARG;
    if (worker < 0 || worker >= ctx->hp.K) return SSD_ERR_ARG;
    if (flags & ~(SSD_FLAG_FIRST | SSD_FLAG_REFRESH | SSD_FLAG_PULL)) return SSD_ERR_ARG;
    if (ctx->hp.delay_k == 0) return SSD_ERR_STATE;
    if (ctx->shared_pre || lacks_device_pre(ctx)) return SSD_ERR_STATE;
    if (!aligned16(grad)) return SSD_ERR_ALIGN;
    if (touches_state(ctx, grad, grad_bytes(ctx))) return SSD_ERR_ARG;
    return launch_glu(ctx, worker, grad, flags, static_cast<cudaStream_t>(cuda_stream));
}

ssd_status ssd_worker_local_step(ssd_ctx *ctx, int32_t worker, const void *grad, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    if (worker < 0 || worker >= ctx->hp.K) return SSD_ERR_ARG;
    int32_t stage, flags;
    schedule_of(ctx, ctx->iter, &stage, &flags);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (stage == SSD_STAGE_WARMUP) {
        if (flags & SSD_FLAG_COPY) return launch_copy(ctx, worker, 1, stream);
        return SSD_OK;
    }
    if (!grad) return SSD_ERR_ARG;
    if (ctx->shared_pre || lacks_device_pre(ctx)) return SSD_ERR_STATE;
    if (!aligned16(grad)) return SSD_ERR_ALIGN;
    if (touches_state(ctx, grad, grad_bytes(ctx))) return SSD_ERR_ARG;
    return launch_glu(ctx, worker, grad, flags, stream);
}

ssd_status ssd_advance(ssd_ctx *ctx)
{
    if (!ctx) return SSD_ERR_ARG;
    advance(ctx);
    return SSD_OK;
}

ssd_status ssd_step(ssd_ctx *ctx, const void *const *grads, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    ssd_status st = check_grads(ctx, grads);
    if (st != SSD_OK) return st;
    int32_t stage, flags;
    schedule_of(ctx, ctx->iter, &stage, &flags);
    if (stage == SSD_STAGE_DELAY && lacks_device_pre(ctx)) return SSD_ERR_STATE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = (stage == SSD_STAGE_WARMUP) ? launch_sync(ctx, grads, flags & SSD_FLAG_COPY, stream)
                                     : launch_step(ctx, grads, flags, stream);
    if (st != SSD_OK) return st;
    advance(ctx);
    return SSD_OK;
}

ssd_status ssd_step_tensors(ssd_ctx *ctx, const void *const *grads, int32_t first_tensor, int32_t num_tensors,
                            void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    ssd_status st = check_grads(ctx, grads);
    if (st != SSD_OK) return st;
    const int32_t T = static_cast<int32_t>(ctx->offsets.size());
    if (first_tensor < 0 || num_tensors < 1 || first_tensor > T - num_tensors) return SSD_ERR_ARG;
    const int64_t lo = ctx->offsets[first_tensor];
    const int64_t hi = first_tensor + num_tensors < T ? ctx->offsets[first_tensor + num_tensors] : ctx->n;
    if (hi == lo) return SSD_OK;                      // only empty tensors
    int32_t stage, flags;
    schedule_of(ctx, ctx->iter, &stage, &flags);
    if (stage == SSD_STAGE_DELAY && lacks_device_pre(ctx)) return SSD_ERR_STATE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    return (stage == SSD_STAGE_WARMUP) ? launch_sync(ctx, grads, flags & SSD_FLAG_COPY, stream, lo, hi - lo)
                                       : launch_step(ctx, grads, flags, stream, lo, hi - lo);
}

ssd_status ssd_step_host(ssd_ctx *ctx, const void *const *host_grads, void *const *staging,
                         float *host_w_out, void *cuda_stream)
{
    if (!ctx || !staging) return SSD_ERR_ARG;
    for (int i = 0; i < ctx->hp.K; ++i) {
        if (!staging[i] || (host_grads && !host_grads[i])) return SSD_ERR_ARG;
        if (!aligned16(staging[i])) return SSD_ERR_ALIGN;
        if (touches_state(ctx, staging[i], grad_bytes(ctx))) return SSD_ERR_ARG;
    }
    int32_t stage, flags;
    schedule_of(ctx, ctx->iter, &stage, &flags);
    const bool glu_stage = stage == SSD_STAGE_DELAY && ctx->hp.local_updater == SSD_LOCAL_GLU;
    if (glu_stage && !ctx->pre_on_device && !ctx->host_pre) return SSD_ERR_STATE;
    ssd_status st = ensure_device(ctx);
    if (st != SSD_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int K = ctx->hp.K;
    const size_t sg = ctx->hp.grad_dtype == SSD_BF16 ? 2 : 4;
    // A host-resident pre_weight travels with the gradients: its slice of a chunk is copied into
    // one of the device slices before the chunk's kernel (not on the first GLU call, which does
    // not read it) and copied back after it on the iterations that overwrite it.
    const bool host_pre = glu_stage && ctx->host_pre;
    // (nor on a pull iteration of a context with merged device weights, which skips the local update)
    const bool pre_in = host_pre && !(flags & SSD_FLAG_FIRST) && !(ctx->merged_dev && (flags & SSD_FLAG_PULL));
    const bool pre_out = host_pre && (flags & (SSD_FLAG_FIRST | SSD_FLAG_REFRESH));
    const int slots = ctx->pre_slots;

    // The arena is cut into chunks; chunk c's inputs are copied in on a side stream while
    // chunk c-1 is being updated on the caller's stream and chunk c-2's results are copied
    // out on a second side stream.  The update is elementwise, so chunks are independent.
    const int64_t chunk = ctx->host_chunk;
    const int chunks = static_cast<int>((ctx->n + chunk - 1) / chunk);
    // events: [2c] chunk c copied in, [2c+1] chunk c updated, then start, end, and one per device
    // slice ("the slice may be overwritten")
    const size_t ev_start_at = 2 * static_cast<size_t>(chunks), ev_end_at = ev_start_at + 1, ev_slot_at = ev_start_at + 2;
    cudaError_t e = cudaSuccess;
    if (!ctx->in_stream) e = cudaStreamCreateWithFlags(&ctx->in_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess && !ctx->out_stream) e = cudaStreamCreateWithFlags(&ctx->out_stream, cudaStreamNonBlocking);
    while (e == cudaSuccess && ctx->events.size() < ev_slot_at + kMaxPreSlots) {
        cudaEvent_t ev;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e == cudaSuccess) ctx->events.push_back(ev);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    cudaEvent_t ev_start = ctx->events[ev_start_at], ev_end = ctx->events[ev_end_at];
    const bool copies_out = host_w_out || pre_out;
    // everything already enqueued on the caller's stream comes first
    e = cudaEventRecord(ev_start, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->in_stream, ev_start, 0);
    if (e == cudaSuccess && copies_out) e = cudaStreamWaitEvent(ctx->out_stream, ev_start, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    for (int c = 0; c < chunks; ++c) {
        const int64_t lo = static_cast<int64_t>(c) * chunk;
        const int64_t count = ctx->n - lo < chunk ? ctx->n - lo : chunk;
        const int slot = host_pre ? c % slots : 0;
        float *slice = host_pre ? ctx->pre_slices + static_cast<int64_t>(slot) * slice_elems(ctx) : nullptr;
        cudaEvent_t ev_slot = ctx->events[ev_slot_at + slot];
        // the slice is free once the chunk that used it last (c - slots) is done with it
        if (host_pre && c >= slots) e = cudaStreamWaitEvent(ctx->in_stream, ev_slot, 0);
        for (int i = 0; host_grads && i < K && e == cudaSuccess; ++i)
            e = cudaMemcpyAsync(static_cast<unsigned char *>(staging[i]) + lo * sg,
                                static_cast<const unsigned char *>(host_grads[i]) + lo * sg, count * sg,
                                cudaMemcpyHostToDevice, ctx->in_stream);
        if (e == cudaSuccess && pre_in)
            e = cudaMemcpyAsync(slice, ctx->host_pre + lo, count * sizeof(float), cudaMemcpyHostToDevice,
                                ctx->in_stream);
        if (e == cudaSuccess) e = cudaEventRecord(ctx->events[2 * c], ctx->in_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->events[2 * c], 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        st = (stage == SSD_STAGE_WARMUP)
                 ? launch_sync(ctx, const_cast<const void *const *>(staging), flags & SSD_FLAG_COPY, stream, lo, count)
                 : launch_step(ctx, const_cast<const void *const *>(staging), flags, stream, lo, count, slice);
        if (st != SSD_OK) return st;
        if (copies_out) {
            e = cudaEventRecord(ctx->events[2 * c + 1], stream);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->out_stream, ctx->events[2 * c + 1], 0);
            if (e == cudaSuccess && host_w_out)
                e = cudaMemcpyAsync(host_w_out + lo, ctx->w + lo, count * sizeof(float), cudaMemcpyDeviceToHost,
                                    ctx->out_stream);
            if (e == cudaSuccess && pre_out)
                e = cudaMemcpyAsync(ctx->host_pre + lo, slice, count * sizeof(float), cudaMemcpyDeviceToHost,
                                    ctx->out_stream);
        }
        if (e == cudaSuccess && host_pre) e = cudaEventRecord(ev_slot, pre_out ? ctx->out_stream : stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    if (copies_out) {
        // the caller's stream ends behind the last copy out
        e = cudaEventRecord(ev_end, ctx->out_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ev_end, 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    advance(ctx);
    return SSD_OK;
}

ssd_status ssd_set_host_chunk(ssd_ctx *ctx, int64_t chunk_elems)
{
    if (!ctx) return SSD_ERR_ARG;
    if (chunk_elems == 0) chunk_elems = kHostChunkElems;
    if (chunk_elems < 1024 || chunk_elems % 1024 != 0 || chunk_elems > (int64_t(1) << 30)) return SSD_ERR_ARG;
    if (ctx->host_pre) return SSD_ERR_STATE;          // the device slices were sized for the current chunk
    ctx->host_chunk = chunk_elems;
    return SSD_OK;
}

ssd_status ssd_set_host_pre_weight(ssd_ctx *ctx, float *host_pre, float *device_slices, int32_t slots)
{
    if (!ctx) return SSD_ERR_ARG;
    if (!host_pre && !device_slices && slots == 0) {       // off again
        ctx->host_pre = ctx->pre_slices = nullptr;
        ctx->pre_slots = 0;
        return SSD_OK;
    }
    if (!host_pre || !device_slices || slots < 1 || slots > kMaxPreSlots) return SSD_ERR_ARG;
    if (!ctx->has_workers || ctx->hp.delay_k == 0 || ctx->pre_on_device) return SSD_ERR_STATE;
    if (!aligned16(host_pre) || !aligned16(device_slices)) return SSD_ERR_ALIGN;
    const size_t bytes = static_cast<size_t>(slots) * static_cast<size_t>(slice_elems(ctx)) * sizeof(float);
    if (touches_state(ctx, device_slices, bytes)) return SSD_ERR_ARG;
    ctx->host_pre = host_pre;
    ctx->pre_slices = device_slices;
    ctx->pre_slots = slots;
    return SSD_OK;
}

ssd_status ssd_broadcast_weights(ssd_ctx *ctx, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    if (!ctx->has_workers) return SSD_ERR_STATE;
    return launch_copy(ctx, 0, ctx->hp.K, static_cast<cudaStream_t>(cuda_stream));
}

ssd_status ssd_worker_weights(const ssd_ctx *ctx, int32_t worker, const float **weights, int32_t *view)
{
    if (!ctx) return SSD_ERR_ARG;
    if (worker < 0 || worker >= ctx->hp.K) return SSD_ERR_ARG;
    int32_t v = SSD_VIEW_GLOBAL;
    if (ctx->iter > 0) {
        int32_t stage, flags;
        schedule_of(ctx, ctx->iter - 1, &stage, &flags);
        if (stage == SSD_STAGE_WARMUP) v = (flags & SSD_FLAG_COPY) ? SSD_VIEW_LOCAL : SSD_VIEW_GLOBAL;
        else v = ((flags & SSD_FLAG_PULL) && !ctx->merged_dev) ? SSD_VIEW_DEVICE : SSD_VIEW_LOCAL;
    }
    if (view) *view = v;
    if (weights)
        *weights = v == SSD_VIEW_GLOBAL ? ctx->w : v == SSD_VIEW_LOCAL ? ctx->w_loc[worker] : ctx->w_dev[worker];
    return SSD_OK;
}

ssd_status ssd_get_counters(const ssd_ctx *ctx, int64_t *iter, int64_t *loc_update,
                            int32_t *next_stage, int32_t *next_flags)
{
    if (!ctx) return SSD_ERR_ARG;
    int32_t stage, flags;
    schedule_of(ctx, ctx->iter, &stage, &flags);
    if (iter) *iter = ctx->iter;
    if (loc_update) *loc_update = ctx->loc_update;
    if (next_stage) *next_stage = stage;
    if (next_flags) *next_flags = flags;
    return SSD_OK;
}

ssd_status ssd_set_counters(ssd_ctx *ctx, int64_t iter, int64_t loc_update)
{
    if (!ctx || iter < 0 || loc_update < 0) return SSD_ERR_ARG;
    int64_t expect = 0;
    if (ctx->hp.delay_k > 0 && iter > ctx->hp.warmup_iters) expect = iter - ctx->hp.warmup_iters;
    if (loc_update != expect) return SSD_ERR_STATE;
    ctx->iter = iter;
    ctx->loc_update = loc_update;
    return SSD_OK;
}

ssd_status ssd_tensor_table_bytes(const ssd_ctx *ctx, int64_t *bytes)
{
    if (!ctx || !bytes) return SSD_ERR_ARG;
    *bytes = static_cast<int64_t>(table_bytes(ctx));
    return SSD_OK;
}

ssd_status ssd_set_tensor_scales(ssd_ctx *ctx, const float *lr_mult, const float *wd_mult,
                                 void *device_table, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    if (!device_table) {                       // back to uniform hyper-parameters
        ctx->tensor_table = nullptr;
        ctx->lr_mult.clear();
        ctx->wd_mult.clear();
        return SSD_OK;
    }
    if (!aligned16(device_table)) return SSD_ERR_ALIGN;
    const size_t T = ctx->offsets.size();
    for (size_t t = 0; t < T; ++t) {
        if (lr_mult && (!(lr_mult[t] > 0.0f) || !std::isfinite(lr_mult[t]))) return SSD_ERR_ARG;
        if (wd_mult && !std::isfinite(wd_mult[t])) return SSD_ERR_ARG;
    }
    std::vector<float> lm(T, 1.0f), wm(T, 1.0f);
    if (lr_mult) lm.assign(lr_mult, lr_mult + T);
    if (wd_mult) wm.assign(wd_mult, wd_mult + T);
    void *old_table = ctx->tensor_table;
    ctx->lr_mult.swap(lm);
    ctx->wd_mult.swap(wm);
    ctx->tensor_table = device_table;
    ssd_status st = upload_table(ctx, static_cast<cudaStream_t>(cuda_stream));
    if (st != SSD_OK) {
        ctx->lr_mult.swap(lm);
        ctx->wd_mult.swap(wm);
        ctx->tensor_table = old_table;
    }
    return st;
}

ssd_status ssd_set_lr(ssd_ctx *ctx, float lr, float lr_local, void *cuda_stream)
{
    if (!ctx) return SSD_ERR_ARG;
    if (!std::isnan(lr) && (!(lr > 0.0f) || !std::isfinite(lr))) return SSD_ERR_ARG;
    if (std::isinf(lr_local)) return SSD_ERR_ARG;
    if (!std::isnan(lr)) {
        ctx->hp.lr = lr;
        ctx->s.lr = lr;
        ctx->s.c = derive_sync_scale(lr, ctx->hp.momentum, ctx->hp.delay_k);
    }
    if (!std::isnan(lr_local)) {
        ctx->hp.lr_local = lr_local;
        ctx->s.lr_loc = lr_local;
    }
    if (ctx->tensor_table) return upload_table(ctx, static_cast<cudaStream_t>(cuda_stream));
    return SSD_OK;
}

ssd_status ssd_get_hparams(const ssd_ctx *ctx, ssd_hparams *resolved, float *sync_scale)
{
    if (!ctx) return SSD_ERR_ARG;
    if (resolved) *resolved = ctx->hp;
    if (sync_scale) *sync_scale = ctx->s.c;
    return SSD_OK;
}

ssd_status ssd_set_launch(ssd_ctx *ctx, int32_t threads_per_block, int32_t blocks_per_sm)
{
    if (!ctx) return SSD_ERR_ARG;
    if (threads_per_block != 0 &&
        (threads_per_block < 64 || threads_per_block > kMaxThreads || threads_per_block % 32 != 0))
        return SSD_ERR_ARG;
    if (blocks_per_sm < 0 || blocks_per_sm > 32) return SSD_ERR_ARG;
    ctx->threads = threads_per_block;
    ctx->blocks_per_sm = blocks_per_sm;
    return SSD_OK;
}

ssd_status ssd_get_launch(const ssd_ctx *ctx, int32_t *threads_per_block, int32_t *blocks_per_sm,
                          int32_t *vector_elems, int32_t *batch)
{
    if (!ctx) return SSD_ERR_ARG;
    if (threads_per_block) *threads_per_block = ctx->threads;
    if (blocks_per_sm) *blocks_per_sm = ctx->blocks_per_sm;
    if (vector_elems) *vector_elems = ctx->force_vw;
    if (batch) *batch = ctx->force_batch;
    return SSD_OK;
}

ssd_status ssd_set_kernel_shape(ssd_ctx *ctx, int32_t vector_elems, int32_t batch)
{
    if (!ctx) return SSD_ERR_ARG;
    if (vector_elems != 0 && vector_elems != 4 && vector_elems != 8 && vector_elems != 16) return SSD_ERR_ARG;
    if (batch != 0 && batch != 1 && batch != 2 && batch != 4 && batch != 8) return SSD_ERR_ARG;
    ctx->force_vw = vector_elems;
    ctx->force_batch = batch;
    return SSD_OK;
}

ssd_status ssd_set_staging(ssd_ctx *ctx, int32_t stages)
{
    if (!ctx) return SSD_ERR_ARG;
    if (stages != 0 && (stages < 2 || stages > kRingMaxStages)) return SSD_ERR_ARG;
    ctx->staging = stages;
    return SSD_OK;
}

ssd_status ssd_staging_error(ssd_ctx *ctx, int32_t *flag)
{
    if (!ctx || !flag) return SSD_ERR_ARG;
    int value = 0;
    cudaError_t e = cudaMemcpyFromSymbol(&value, g_ring_error, sizeof value);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    *flag = value;
    return SSD_OK;
}

int64_t ssd_kernel_launches(const ssd_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *ssd_status_str(ssd_status status)
{
    switch (status) {
    case SSD_OK: return "ok";
    case SSD_ERR_ARG: return "invalid argument";
    case SSD_ERR_ALIGN: return "device pointer not 16-byte aligned";
    case SSD_ERR_LAYOUT: return "invalid parameter layout";
    case SSD_ERR_STATE: return "call not valid in the context's current stage or mode";
    case SSD_ERR_CUDA: return "CUDA runtime error";
    case SSD_ERR_NOMEM: return "out of host memory";
    case SSD_ERR_TOO_LARGE: return "more tensors than the static table holds (SSD_STATIC_TABLE_MAX_TENSORS)";
    }
    return "unknown status";
}

const char *ssd_last_cuda_error(const ssd_ctx *ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

}  // extern "C"
