// C ABI and host-side protocol state of the n-softsync parameter server
// (arXiv 1511.05950, Section 2.1-2.4).  The O(N) work is in update_kernels.cuh;
// this file keeps the scalar timestamp clock, computes staleness at push time,
// groups gradients first come first grouped, builds the per-launch scale table
// and records what it decided in the update log.
#include "../../include/softsync_ps.h"
#include "update_kernels.cuh"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <deque>
#include <mutex>
#include <new>
#include <unordered_set>
#include <vector>

namespace {

using softsync::BulkPlan;
using softsync::BulkStatus;
using softsync::GradBf16;
using softsync::GradFp32;
using softsync::LaunchParams;

struct Entry {                 // one pushed gradient waiting for its update
    int32_t learner;
    int64_t push_index, ts_grad, tau, sigma;
    float alpha0;              // base rate in force when the gradient arrived
    const void *grad;
    int slot;                  // staging slot it occupies, -1 if borrowed from the caller
    bool by_learner;           // the slot was lent to a learner (ps_push_slot): its producer may be a kernel
};

struct TimedLaunch { cudaEvent_t start, stop; };
constexpr size_t kMaxTimedLaunches = 1 << 16;   // launches held between two ps_kernel_time calls

}  // namespace

struct ps_ctx {
    int64_t n = 0;
    int lambda = 0, split = 0, c = 0, modulation = 0;
    float alpha0 = 0, momentum = 0, weight_decay = 0;
    float penalty_base = 0.5f;             // rho of PS_MOD_EXP_STALENESS
    int device = 0;

    int num_layers = 0;                    // per-layer multipliers (0: none)
    int64_t layer_end[PS_MAX_LAYERS] = {};
    float layer_lr[PS_MAX_LAYERS] = {}, layer_wd[PS_MAX_LAYERS] = {};

    float *w = nullptr, *v = nullptr;
    unsigned short *mirror = nullptr;      // optional caller-owned bf16 copy of theta
    int num_replicas = 0;                  // optional caller-owned fp32 copies of theta (ps_bind_weight_replicas)
    float *replicas[PS_MAX_REPLICAS] = {};
    char *staging = nullptr;
    int64_t slot_bytes = 0;
    std::vector<int> free_slots;
    std::vector<char> slot_lent;           // 1 while a learner holds the slot between acquire and push
    std::vector<cudaEvent_t> slot_consumed;  // recorded behind the update kernel that read the slot last (lazily created)
    std::vector<char> slot_has_consumer;
    std::vector<cudaEvent_t> slot_filled;    // recorded on a learner's stream by ps_slot_written (lazily created)
    int num_slots = 0;

    int grad_dtype = PS_GRAD_FP32;
    int fuse_t = 1;
    cudaStream_t stream = nullptr;
    int64_t queue_groups = 64;
    int64_t log_updates = 65536;           // set in ps_create: about one million log entries
    int timing = 0, kernel_choice = PS_KERNEL_AUTO, block_threads = 0, overlap_launch = 0;
    int protocol = PS_PROTOCOL_SOFTSYNC;
    int zigzag = 1;
    int sm_count = 0;

    int bulk_tile = 0, bulk_stages = 2, bulk_wait_limit = 1 << 20, bulk_selftest = 0;
    BulkStatus *bulk_status = nullptr;     // pinned, device-mapped host memory (allocated by the first bulk launch)
    bool bulk_attr_set[2][2] = {};         // dynamic shared-memory opt-in done, per (dtype, layers) instantiation

    int64_t ts_applied = 0;                // updates whose kernel has been enqueued
    int64_t launches = 0;                  // update kernels enqueued so far
    int last_kernel = 0;                   // ps_kernel_choice of the most recent launch
    int64_t launches_by_kind[4] = {};      // indexed by ps_kernel_choice
    std::deque<std::vector<Entry>> ready;  // complete groups, oldest first
    std::vector<Entry> filling;            // the group being collected (< c entries)
    std::vector<int64_t> push_count;       // per learner

    std::deque<ps_log_entry> log;          // c entries per update, oldest first
    int64_t log_first_update = 0;

    std::vector<TimedLaunch> timed, spare_events;
    int last_cuda_error = 0;

    // asynchronous weight read-back: a second stream so that a device-to-host copy of theta can run
    // while the next gradients are still arriving host-to-device on the main stream
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t weights_ready = nullptr, weights_copied = nullptr;
    bool copy_in_flight = false;
};

namespace {

std::mutex g_live_mutex;
std::unordered_set<ps_ctx *> g_live;       // handles that ps_create returned and ps_destroy has not seen

bool is_live(ps_ctx *ps)
{
    if (!ps) return false;
    std::lock_guard<std::mutex> lock(g_live_mutex);
    return g_live.count(ps) != 0;
}

int cuda_fail(ps_ctx *ps, cudaError_t e)
{
    ps->last_cuda_error = static_cast<int>(e);
    return PS_ERR_CUDA;
}
// No exception may cross the C boundary: allocation failures become PS_ERR_NOMEM.
#define PS_CATCH_ALL catch (const std::bad_alloc &) { return PS_ERR_NOMEM; } catch (...) { return PS_ERR_INVALID_ARG; }
#define PS_CUDA(ps, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail((ps), e_); } while (0)

// Makes the server's GPU current for the duration of a call and restores the caller's choice afterwards,
// so that a process driving several GPUs may call any handle at any time.
class DeviceGuard {
public:
    explicit DeviceGuard(const ps_ctx *ps)
    {
        if (ps->device >= 0 && cudaGetDevice(&prev_) == cudaSuccess && prev_ != ps->device)
            switched_ = cudaSetDevice(ps->device) == cudaSuccess;
    }
    ~DeviceGuard() { if (switched_) cudaSetDevice(prev_); }
    DeviceGuard(const DeviceGuard &) = delete;
    DeviceGuard &operator=(const DeviceGuard &) = delete;
private:
    int prev_ = -1;
    bool switched_ = false;
};

size_t grad_elem_bytes(const ps_ctx *ps) { return ps->grad_dtype == PS_GRAD_BF16 ? 2 : 4; }

int64_t ts_logical(const ps_ctx *ps) { return ps->ts_applied + static_cast<int64_t>(ps->ready.size()); }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Summation order inside a group: ascending learner id, then push index.
bool entry_before(const Entry &a, const Entry &b)
{
    return a.learner != b.learner ? a.learner < b.learner : a.push_index < b.push_index;
}

constexpr int kChunk = 8;            // gradient loads in flight per thread beyond the first EC
constexpr int kHead = 16;            // largest compile-time first chunk of gradient loads
constexpr int kBulkThreads = 512;

template <bool LAYERS> constexpr int seg_capacity() { return LAYERS ? PS_MAX_LAYERS : 1; }
template <int MAXE, bool LAYERS> using Params = LaunchParams<MAXE, seg_capacity<LAYERS>()>;

template <typename GT, int VEC, int EC, bool MORE, bool LAYERS, int MAXE, int CT = 0>
cudaError_t launch_variant(const Params<MAXE, LAYERS> &p, int blocks, int threads, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(static_cast<unsigned>(threads));
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, softsync::softsync_update_kernel<GT, VEC, EC, MORE, kChunk, LAYERS, MAXE, seg_capacity<LAYERS>(), CT>, p);
}

// E = T*c <= HEAD: the straight-line instantiation with exactly E loads up front.
template <typename GT, int VEC, int HEAD, bool LAYERS, int MAXE, int EC = HEAD>
cudaError_t launch_exact(int E, const Params<MAXE, LAYERS> &p, int blocks, int threads, cudaStream_t stream)
{
    if constexpr (EC == 0) {
        return cudaErrorInvalidValue;
    } else {
        if (E == EC) {
            // c = 1 (every gradient its own update, the fused asynchronous case) has its own instantiation
            if constexpr (!LAYERS)
                if (p.c == 1) return launch_variant<GT, VEC, EC, false, LAYERS, MAXE, 1>(p, blocks, threads, stream);
            return launch_variant<GT, VEC, EC, false, LAYERS, MAXE>(p, blocks, threads, stream);
        }
        return launch_exact<GT, VEC, HEAD, LAYERS, MAXE, EC - 1>(E, p, blocks, threads, stream);
    }
}

template <typename GT, int VEC, int HEAD, bool LAYERS, int MAXE>
cudaError_t launch_vector(int E, const Params<MAXE, LAYERS> &p, int blocks, int threads, cudaStream_t stream)
{
    if constexpr (MAXE <= HEAD) {                        // the small parameter block: T*c <= HEAD always
        return launch_exact<GT, VEC, MAXE, LAYERS, MAXE>(E, p, blocks, threads, stream);
    } else {
        if (E <= HEAD) return cudaErrorInvalidValue;     // such launches use the small parameter block
    }
    return launch_variant<GT, VEC, HEAD, true, LAYERS, MAXE>(p, blocks, threads, stream);   // HEAD loads, then chunks
}

// Launch shape of the bulk-copy kernel.  Measured on the 61 M-element configurations, few large tiles win:
// two stages whose tiles fill most of an SM's shared memory (one block per SM) run 8-25 % faster than four
// stages of quarter-size tiles (two blocks per SM), because every tile costs a block-wide barrier and one
// thread's round of copy instructions.
struct BulkShape { int tile; size_t smem; int threads; int blocks_per_sm; };

BulkShape bulk_shape(int entries, int grad_bytes, int stages, int tile_option, int threads_option)
{
    const size_t per_elem = 8 + static_cast<size_t>(entries) * grad_bytes;
    const size_t limit = 200 * 1024;                     // of the 227 KB one block may take
    int tile = tile_option ? tile_option : 8192;         // halved until the stages of one block fit
    while (tile > 256 && static_cast<size_t>(stages) * tile * per_elem > limit) tile >>= 1;
    BulkShape sh;
    sh.tile = tile;
    sh.smem = static_cast<size_t>(stages) * tile * per_elem;
    sh.threads = threads_option ? threads_option : kBulkThreads;
    const size_t per_sm = 227 * 1024;
    const int by_smem = static_cast<int>(std::max<size_t>(1, per_sm / (sh.smem + 1024)));
    sh.blocks_per_sm = std::max(1, std::min(by_smem, 2048 / sh.threads));
    return sh;
}

template <typename GT, bool LAYERS, int MAXE>
cudaError_t launch_bulk(ps_ctx *ps, const Params<MAXE, LAYERS> &p)
{
    constexpr int kSeg = seg_capacity<LAYERS>();
    const int gb = ps->grad_dtype == PS_GRAD_BF16 ? 2 : 4;
    const int stages = ps->bulk_stages;
    const BulkShape sh = bulk_shape(p.T * p.c, gb, stages, ps->bulk_tile, ps->block_threads);
    const int tile = sh.tile;
    const size_t smem = sh.smem;
    if (smem > 220 * 1024) return cudaErrorInvalidConfiguration;
    auto kernel = softsync::softsync_update_bulk_kernel<GT, LAYERS, MAXE, kSeg>;
    bool &attr_set = ps->bulk_attr_set[gb == 2][LAYERS];
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (!ps->bulk_status) {
        cudaError_t e = cudaHostAlloc(reinterpret_cast<void **>(&ps->bulk_status), 64, cudaHostAllocMapped);
        if (e != cudaSuccess) return e;
        std::memset(ps->bulk_status, 0, 64);
    }
    BulkPlan plan;
    plan.tile_elems = tile;
    plan.ntiles = p.n / tile;
    plan.stages = stages;
    plan.wait_limit = ps->bulk_wait_limit;
    plan.selftest = ps->bulk_selftest;
    ps->bulk_selftest = 0;
    cudaError_t e = cudaHostGetDevicePointer(reinterpret_cast<void **>(&plan.status), ps->bulk_status, 0);
    if (e != cudaSuccess) return e;
    const int threads = sh.threads;
    const long long cap = static_cast<long long>(ps->sm_count) * sh.blocks_per_sm;
    const int blocks = static_cast<int>(std::max<long long>(1, std::min<long long>(plan.ntiles, cap)));

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(static_cast<unsigned>(threads));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = ps->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p, plan);
}

enum LaunchKind { kScalar = PS_KERNEL_SCALAR, kVector = PS_KERNEL_VECTOR, kBulk = PS_KERNEL_BULK };

template <int MAXE, bool LAYERS>
cudaError_t launch_update(ps_ctx *ps, const Params<MAXE, LAYERS> &p, int kind)
{
    const bool bf16 = ps->grad_dtype == PS_GRAD_BF16;
    if (kind == kBulk) {
        if constexpr (MAXE <= kHead) {
            return bf16 ? launch_bulk<GradBf16, LAYERS, MAXE>(ps, p) : launch_bulk<GradFp32, LAYERS, MAXE>(ps, p);
        } else {
            return cudaErrorInvalidValue;                // checked by the caller: T*c <= 16 only
        }
    }
    const int vec = kind == kVector ? 4 : 1;
    const int threads = ps->block_threads ? ps->block_threads : 128;
    const long long frags = std::max<long long>(1, (p.n + vec - 1) / vec);
    const long long blocks = (frags + threads - 1) / threads;    // one fragment per thread
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int b = static_cast<int>(blocks);
    const int E = p.T * p.c;
    if (kind == kScalar)
        return bf16 ? launch_variant<GradBf16, 1, 0, true, LAYERS, MAXE>(p, b, threads, ps->stream)
                    : launch_variant<GradFp32, 1, 0, true, LAYERS, MAXE>(p, b, threads, ps->stream);
    return bf16 ? launch_vector<GradBf16, 4, kHead, LAYERS, MAXE>(E, p, b, threads, ps->stream)
                : launch_vector<GradFp32, 4, kHead, LAYERS, MAXE>(E, p, b, threads, ps->stream);
}

bool aligned_to(const void *p, uintptr_t bytes) { return (reinterpret_cast<uintptr_t>(p) & (bytes - 1)) == 0; }

// Fills the scale table of one launch (Eq. 3 folded with the 1/c of Eq. 2) for the `T`
// oldest complete groups and the log entries that describe them.  vector_ok / bulk_ok: whether every
// pointer of the launch is aligned for the widths those kernels use.
template <int MAXE, bool LAYERS>
void build_launch(ps_ctx *ps, int T, Params<MAXE, LAYERS> &p, std::vector<ps_log_entry> &entries,
                  bool &vector_ok, bool &bulk_ok)
{
    p.w = ps->w; p.v = ps->v; p.n = ps->n;
    p.momentum = make_float2(ps->momentum, ps->momentum); p.T = T; p.c = ps->c;
    p.overlap = ps->overlap_launch;
    p.reverse = ps->zigzag ? static_cast<int>(ps->launches & 1) : 0;   // zig-zag over the vector from launch to launch
    p.mirror = ps->mirror;
    p.nrep = ps->num_replicas;
    for (int r = 0; r < ps->num_replicas; ++r) p.rep[r] = ps->replicas[r];
    p.layers.count = 0;
    if constexpr (LAYERS) {
        p.layers.count = ps->num_layers;
        for (int q = 0; q < ps->num_layers; ++q) {
            p.layers.end[q] = ps->layer_end[q]; p.layers.lm[q] = ps->layer_lr[q]; p.layers.dm[q] = ps->layer_wd[q];
        }
    }
    // the vector kernel moves theta and v in 16-byte pieces, fp32 gradients too; bf16 gradients and the
    // bf16 mirror in 8-byte pieces.  The bulk copies need 16 bytes everywhere.
    const uintptr_t grad_align = ps->grad_dtype == PS_GRAD_BF16 ? 8 : 16;
    vector_ok = aligned16(ps->w) && aligned16(ps->v) && aligned_to(ps->mirror, 8);
    for (int r = 0; r < ps->num_replicas; ++r) vector_ok = vector_ok && aligned16(ps->replicas[r]);
    bulk_ok = vector_ok;
    const double wd = static_cast<double>(ps->weight_decay);
    for (int t = 0; t < T; ++t) {
        std::vector<Entry> &grp = ps->ready[t];
        std::stable_sort(grp.begin(), grp.end(), entry_before);
        double sum = 0.0;
        for (int l = 0; l < ps->c; ++l) {
            const Entry &en = grp[l];
            double step;
            if (ps->modulation == PS_MOD_EXP_STALENESS)      // alpha0 * rho^tau, then the 1/c of Eq. 2
                step = static_cast<double>(en.alpha0) * std::pow(static_cast<double>(ps->penalty_base), static_cast<double>(en.tau)) /
                       static_cast<double>(ps->c);
            else                                             // Eq. 3 (sigma = 1 for the constant rate)
                step = static_cast<double>(en.alpha0) / (static_cast<double>(ps->c) * static_cast<double>(en.sigma));
            const float s = static_cast<float>(step);
            p.s[t * ps->c + l] = make_float2(s, s);
            p.g[t * ps->c + l] = en.grad;
            vector_ok = vector_ok && aligned_to(en.grad, grad_align);
            bulk_ok = bulk_ok && aligned16(en.grad);
            if (en.by_learner) p.overlap = 0;               // its producer may be the kernel directly before this one
            sum += static_cast<double>(s);
        }
        const float d = static_cast<float>(wd * sum);   // every gradient carries + wd * theta
        p.d[t] = make_float2(d, d);
        for (int l = 0; l < ps->c; ++l) {
            const Entry &en = grp[l];
            ps_log_entry le;
            le.update = ps->ts_applied + t;
            le.push_index = en.push_index; le.ts_grad = en.ts_grad; le.tau = en.tau; le.sigma = en.sigma;
            le.learner = en.learner; le.position = l;
            le.scale = p.s[t * ps->c + l].x; le.decay = d;
            entries.push_back(le);
        }
    }
}

// theta may not be overwritten while an asynchronous read-back is still reading it.
int order_after_readback(ps_ctx *ps)
{
    if (ps->copy_in_flight) {
        PS_CUDA(ps, cudaStreamWaitEvent(ps->stream, ps->weights_copied, 0));
        ps->copy_in_flight = false;
    }
    return PS_OK;
}

// Rewrites the bf16 mirror and the fp32 replicas from theta (set-up paths; updates keep them current themselves).
int refresh_mirror(ps_ctx *ps)
{
    if (!ps->w || ps->n == 0) return PS_OK;
    for (int r = 0; r < ps->num_replicas; ++r)
        PS_CUDA(ps, cudaMemcpyAsync(ps->replicas[r], ps->w, static_cast<size_t>(ps->n) * sizeof(float),
                                    cudaMemcpyDefault, ps->stream));
    if (!ps->mirror) return PS_OK;
    const int threads = 256;
    const long long want = (ps->n + threads - 1) / threads;
    const int blocks = static_cast<int>(std::min<long long>(want, static_cast<long long>(ps->sm_count) * 32));
    softsync::mirror_kernel<<<blocks, threads, 0, ps->stream>>>(ps->w, ps->mirror, ps->n);
    PS_CUDA(ps, cudaGetLastError());
    return PS_OK;
}

int take_events(ps_ctx *ps, TimedLaunch &tl)
{
    if (!ps->spare_events.empty()) { tl = ps->spare_events.back(); ps->spare_events.pop_back(); return PS_OK; }
    PS_CUDA(ps, cudaEventCreate(&tl.start));
    PS_CUDA(ps, cudaEventCreate(&tl.stop));
    return PS_OK;
}

template <int MAXE, bool LAYERS>
int apply_groups(ps_ctx *ps, int T)
{
    Params<MAXE, LAYERS> p;
    std::vector<ps_log_entry> entries;
    entries.reserve(static_cast<size_t>(T) * ps->c);
    bool vector_ok = false, bulk_ok = false;
    build_launch<MAXE, LAYERS>(ps, T, p, entries, vector_ok, bulk_ok);
    int kind = vector_ok ? kVector : kScalar;
    if (ps->kernel_choice == PS_KERNEL_SCALAR) kind = kScalar;
    if (ps->kernel_choice == PS_KERNEL_VECTOR && !vector_ok) return PS_ERR_INVALID_ARG;
    if (ps->kernel_choice == PS_KERNEL_BULK) {
        if (!bulk_ok || T * ps->c > kHead) return PS_ERR_INVALID_ARG;
        kind = kBulk;
    }

    if (ps->n > 0) {
        const int rb = order_after_readback(ps);
        if (rb != PS_OK) return rb;
        TimedLaunch tl{};
        const bool timed = ps->timing && ps->timed.size() < kMaxTimedLaunches;
        if (timed) {
            int rc = take_events(ps, tl);
            if (rc != PS_OK) return rc;
            PS_CUDA(ps, cudaEventRecord(tl.start, ps->stream));
        }
        PS_CUDA(ps, (launch_update<MAXE, LAYERS>(ps, p, kind)));
        if (timed) {
            PS_CUDA(ps, cudaEventRecord(tl.stop, ps->stream));
            ps->timed.push_back(tl);
        }
        // a recycled slot may be handed out while this kernel still reads it: remember where the kernel ends
        for (int t = 0; t < T; ++t)
            for (const Entry &en : ps->ready[t])
                if (en.slot >= 0) {
                    if (!ps->slot_consumed[en.slot])
                        PS_CUDA(ps, cudaEventCreateWithFlags(&ps->slot_consumed[en.slot], cudaEventDisableTiming));
                    PS_CUDA(ps, cudaEventRecord(ps->slot_consumed[en.slot], ps->stream));
                    ps->slot_has_consumer[en.slot] = 1;
                }
        ps->last_kernel = kind;
        ps->launches_by_kind[kind] += 1;
    }
    ps->launches += 1;
    // the launch is enqueued: advance the clock, release slots, publish the log
    for (int t = 0; t < T; ++t) {
        for (const Entry &en : ps->ready.front())
            if (en.slot >= 0) ps->free_slots.push_back(en.slot);
        ps->ready.pop_front();
    }
    ps->ts_applied += T;
    for (const ps_log_entry &le : entries) ps->log.push_back(le);
    const int64_t held = static_cast<int64_t>(ps->log.size()) / ps->c;
    if (held > ps->log_updates) {
        const int64_t drop = held - ps->log_updates;
        ps->log.erase(ps->log.begin(), ps->log.begin() + drop * ps->c);
        ps->log_first_update += drop;
    }
    return T;
}

int apply_some(ps_ctx *ps)
{
    if (ps->n > 0 && (!ps->w || !ps->v)) return PS_ERR_NO_STATE;
    if (ps->ready.empty()) return PS_ERR_NOT_READY;
    int T = static_cast<int>(std::min<int64_t>(ps->fuse_t, static_cast<int64_t>(ps->ready.size())));
    T = std::min(T, std::max(1, PS_MAX_ENTRIES / ps->c));
    const bool small = T * ps->c <= kHead;
    if (ps->num_layers > 0)
        return small ? apply_groups<kHead, true>(ps, T) : apply_groups<PS_MAX_ENTRIES, true>(ps, T);
    return small ? apply_groups<kHead, false>(ps, T) : apply_groups<PS_MAX_ENTRIES, false>(ps, T);
}

int push_common(ps_ctx *ps, int learner, const void *grad_dev, int64_t ts, int slot, bool by_learner = false)
{
    const int64_t i = ts_logical(ps);
    Entry en;
    en.learner = learner;
    en.push_index = ps->push_count[learner];
    en.ts_grad = ts;
    en.tau = i - ts;                                      // staleness (Section 2.1)
    en.sigma = 1;                                         // constant rate
    if (ps->modulation == PS_MOD_INV_STALENESS) en.sigma = std::max<int64_t>(en.tau, 1);   // Eq. 3; alpha0 at tau = 0
    if (ps->modulation == PS_MOD_EXP_STALENESS) en.sigma = en.tau;                          // the penalty's exponent
    en.alpha0 = ps->alpha0;
    en.grad = grad_dev;
    en.slot = slot;
    en.by_learner = by_learner;
    ps->push_count[learner] += 1;
    ps->filling.push_back(en);
    if (static_cast<int>(ps->filling.size()) == ps->c) {  // group of c complete: the clock moves on
        ps->ready.push_back(std::move(ps->filling));
        ps->filling.clear();
        ps->filling.reserve(ps->c);
        return PS_READY;
    }
    return PS_OK;
}

int check_push(ps_ctx *ps, int learner, const void *grad, int64_t ts)
{
    if (!grad && ps->n > 0) return PS_ERR_INVALID_ARG;    // a zero-length gradient has no address
    if (learner < 0 || learner >= ps->lambda) return PS_ERR_BAD_LEARNER;
    if (ts < 0 || ts > ts_logical(ps)) return PS_ERR_BAD_TIMESTAMP;
    if (ps->protocol == PS_PROTOCOL_HARDSYNC) {           // Section 2.2: everybody works on the current weights
        if (ts != ts_logical(ps)) return PS_ERR_BAD_TIMESTAMP;
        for (const Entry &en : ps->filling)
            if (en.learner == learner) return PS_ERR_BARRIER;
    }
    if (static_cast<int64_t>(ps->ready.size()) >= ps->queue_groups) return PS_ERR_QUEUE_FULL;
    return PS_OK;
}

void release_events(ps_ctx *ps)
{
    for (auto &tl : ps->timed) ps->spare_events.push_back(tl);
    ps->timed.clear();
}

}  // namespace

extern "C" {

int ps_create(ps_t **out, int64_t num_params, int lambda, int n,
              float alpha0, float momentum, float weight_decay, int modulation)
{
    try {
        if (!out) return PS_ERR_INVALID_ARG;
        *out = nullptr;
        if (num_params < 0 || lambda < 1 || n < 1 || n > lambda) return PS_ERR_INVALID_ARG;
        if (modulation < PS_MOD_CONSTANT || modulation > PS_MOD_EXP_STALENESS) return PS_ERR_INVALID_ARG;
        if (lambda / n > PS_MAX_GROUP) return PS_ERR_INVALID_ARG;
        if (!(alpha0 == alpha0) || !(momentum == momentum) || !(weight_decay == weight_decay)) return PS_ERR_INVALID_ARG;
        ps_ctx *ps = new (std::nothrow) ps_ctx;
        if (!ps) return PS_ERR_NOMEM;
        ps->n = num_params; ps->lambda = lambda; ps->split = n; ps->c = lambda / n;   // Eq. 2: c = floor(lambda / n)
        ps->alpha0 = alpha0; ps->momentum = momentum; ps->weight_decay = weight_decay;
        ps->modulation = modulation;
        ps->log_updates = std::max<int64_t>(1024, (int64_t{1} << 20) / ps->c);
        cudaError_t e = cudaGetDevice(&ps->device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ps->sm_count, cudaDevAttrMultiProcessorCount, ps->device);
        if (e != cudaSuccess) {
            // No usable GPU and there is no CPU path: only a server with zero parameters
            // (protocol bookkeeping alone, nothing to launch) may exist without one.
            cudaGetLastError();
            if (num_params > 0) { delete ps; return PS_ERR_CUDA; }
            ps->device = -1; ps->sm_count = 1;
        }
        try {
            ps->push_count.assign(lambda, 0);
            ps->filling.reserve(ps->c);
        } catch (const std::bad_alloc &) { delete ps; return PS_ERR_NOMEM; }
        {
            std::lock_guard<std::mutex> lock(g_live_mutex);
            g_live.insert(ps);
        }
        *out = ps;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_destroy(ps_t *ps)
{
    try {
        {
            std::lock_guard<std::mutex> lock(g_live_mutex);
            if (!ps || !g_live.erase(ps)) return PS_ERR_INVALID_ARG;
        }
        DeviceGuard on_device(ps);
        if (ps->device >= 0) cudaStreamSynchronize(ps->stream);
        if (ps->copy_stream) {
            cudaStreamSynchronize(ps->copy_stream);
            cudaEventDestroy(ps->weights_ready); cudaEventDestroy(ps->weights_copied);
            cudaStreamDestroy(ps->copy_stream);
        }
        release_events(ps);
        for (auto &tl : ps->spare_events) { cudaEventDestroy(tl.start); cudaEventDestroy(tl.stop); }
        for (cudaEvent_t ev : ps->slot_consumed) if (ev) cudaEventDestroy(ev);
        for (cudaEvent_t ev : ps->slot_filled) if (ev) cudaEventDestroy(ev);
        if (ps->bulk_status) cudaFreeHost(ps->bulk_status);
        delete ps;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_bind_state(ps_t *ps, float *w_dev, float *v_dev)
{
    try {
        if (!is_live(ps) || !w_dev || !v_dev || w_dev == v_dev) return PS_ERR_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(w_dev) & 3u) || (reinterpret_cast<uintptr_t>(v_dev) & 3u)) return PS_ERR_INVALID_ARG;
        {
            const uintptr_t a = reinterpret_cast<uintptr_t>(w_dev), b = reinterpret_cast<uintptr_t>(v_dev);
            const uintptr_t bytes = static_cast<uintptr_t>(ps->n) * sizeof(float);
            if ((a < b ? b - a : a - b) < bytes) return PS_ERR_INVALID_ARG;          // the two ranges overlap
        }
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
        if (w_dev == reinterpret_cast<float *>(ps->mirror) || v_dev == reinterpret_cast<float *>(ps->mirror))
            return PS_ERR_INVALID_ARG;
        for (int r = 0; r < ps->num_replicas; ++r) {                                   // nor a replica bound earlier
            const uintptr_t bytes = static_cast<uintptr_t>(ps->n) * sizeof(float);
            const uintptr_t q = reinterpret_cast<uintptr_t>(ps->replicas[r]);
            for (const float *mine : {w_dev, v_dev}) {
                const uintptr_t a = reinterpret_cast<uintptr_t>(mine);
                if ((a < q ? q - a : a - q) < bytes) return PS_ERR_INVALID_ARG;
            }
        }
        ps->w = w_dev; ps->v = v_dev;
        DeviceGuard on_device(ps);
        return refresh_mirror(ps);                        // a mirror and replicas bound earlier follow the new theta
    } PS_CATCH_ALL
}

int ps_init_weights(ps_t *ps, const float *w_src, int src_is_host)
{
    try {
        if (!is_live(ps) || (!w_src && ps->n > 0)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (ps->n > 0 && (!ps->w || !ps->v)) return PS_ERR_NO_STATE;
        const size_t bytes = static_cast<size_t>(ps->n) * sizeof(float);
        if (bytes) {
            const int rb = order_after_readback(ps);
            if (rb != PS_OK) return rb;
            PS_CUDA(ps, cudaMemcpyAsync(ps->w, w_src, bytes, src_is_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, ps->stream));
            PS_CUDA(ps, cudaMemsetAsync(ps->v, 0, bytes, ps->stream));
            const int rm = refresh_mirror(ps);
            if (rm != PS_OK) return rm;
            if (src_is_host) PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
        }
        for (auto &grp : ps->ready) for (const Entry &en : grp) if (en.slot >= 0) ps->free_slots.push_back(en.slot);
        for (const Entry &en : ps->filling) if (en.slot >= 0) ps->free_slots.push_back(en.slot);
        ps->ready.clear(); ps->filling.clear();
        std::fill(ps->push_count.begin(), ps->push_count.end(), 0);
        ps->ts_applied = 0;
        ps->log.clear(); ps->log_first_update = 0;
        if (ps->bulk_status && ps->bulk_status->code != 0) {
            PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
            std::memset(ps->bulk_status, 0, sizeof(BulkStatus));
        }
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_bind_weight_mirror(ps_t *ps, void *mirror_dev)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (reinterpret_cast<uintptr_t>(mirror_dev) & 1u) return PS_ERR_INVALID_ARG;
        if (mirror_dev && (mirror_dev == ps->w || mirror_dev == ps->v)) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty()) return PS_ERR_INVALID_ARG;               // apply or flush first
        ps->mirror = static_cast<unsigned short *>(mirror_dev);
        return refresh_mirror(ps);
    } PS_CATCH_ALL
}

int ps_bind_weight_replicas(ps_t *ps, int count, float *const *replicas_dev)
{
    try {
        if (!is_live(ps) || count < 0 || count > PS_MAX_REPLICAS || (count > 0 && !replicas_dev)) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty()) return PS_ERR_INVALID_ARG;               // apply or flush first
        const uintptr_t bytes = static_cast<uintptr_t>(ps->n) * sizeof(float);
        for (int r = 0; r < count; ++r) {
            const uintptr_t a = reinterpret_cast<uintptr_t>(replicas_dev[r]);
            if (!a || (a & 3u)) return PS_ERR_INVALID_ARG;
            for (const void *other : {static_cast<const void *>(ps->w), static_cast<const void *>(ps->v)}) {
                const uintptr_t b = reinterpret_cast<uintptr_t>(other);
                if (b && (a < b ? b - a : a - b) < bytes) return PS_ERR_INVALID_ARG;     // overlaps theta or v
            }
            for (int q = 0; q < r; ++q) {                                                // or another replica
                const uintptr_t b = reinterpret_cast<uintptr_t>(replicas_dev[q]);
                if ((a < b ? b - a : a - b) < bytes) return PS_ERR_INVALID_ARG;
            }
            if (const uintptr_t m = reinterpret_cast<uintptr_t>(ps->mirror))             // or the bf16 mirror
                if (a < m ? m - a < bytes : a - m < bytes / 2) return PS_ERR_INVALID_ARG;
        }
        DeviceGuard on_device(ps);
        ps->num_replicas = count;
        for (int r = 0; r < count; ++r) ps->replicas[r] = replicas_dev[r];
        return refresh_mirror(ps);
    } PS_CATCH_ALL
}

int ps_bind_staging(ps_t *ps, void *slots_dev, int64_t slot_bytes, int num_slots)
{
    try {
        if (!is_live(ps) || !slots_dev || num_slots < 1 || slot_bytes < 0) return PS_ERR_INVALID_ARG;
        if (!aligned16(slots_dev) || (slot_bytes & 15)) return PS_ERR_INVALID_ARG;
        if (slot_bytes < ps->n * static_cast<int64_t>(grad_elem_bytes(ps))) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
        ps->staging = static_cast<char *>(slots_dev);
        ps->slot_bytes = slot_bytes; ps->num_slots = num_slots;
        ps->free_slots.clear();
        for (int s = num_slots - 1; s >= 0; --s) ps->free_slots.push_back(s);
        ps->slot_lent.assign(num_slots, 0);
        DeviceGuard on_device(ps);
        for (cudaEvent_t ev : ps->slot_consumed) if (ev) cudaEventDestroy(ev);
        for (cudaEvent_t ev : ps->slot_filled) if (ev) cudaEventDestroy(ev);
        ps->slot_consumed.assign(num_slots, nullptr);
        ps->slot_filled.assign(num_slots, nullptr);
        ps->slot_has_consumer.assign(num_slots, 0);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_set_option(ps_t *ps, int key, int64_t value)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        switch (key) {
        case PS_OPT_GRAD_DTYPE:
            if (value != PS_GRAD_FP32 && value != PS_GRAD_BF16) return PS_ERR_INVALID_ARG;
            if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
            if (ps->staging && ps->slot_bytes < ps->n * (value == PS_GRAD_BF16 ? 2 : 4)) return PS_ERR_INVALID_ARG;
            ps->grad_dtype = static_cast<int>(value); return PS_OK;
        case PS_OPT_FUSE_T:
            if (value < 1 || value > PS_MAX_FUSE_T) return PS_ERR_INVALID_ARG;
            ps->fuse_t = static_cast<int>(value); return PS_OK;
        case PS_OPT_STREAM: {
            if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
            cudaStream_t next = reinterpret_cast<cudaStream_t>(static_cast<uintptr_t>(value));
            if (next != ps->stream && ps->device >= 0 && ps->launches > 0) {
                // updates and copies already enqueued on the old stream come first
                DeviceGuard on_device(ps);
                cudaEvent_t ev;
                PS_CUDA(ps, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
                cudaError_t e = cudaEventRecord(ev, ps->stream);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(next, ev, 0);
                cudaEventDestroy(ev);
                if (e != cudaSuccess) return cuda_fail(ps, e);
            }
            ps->stream = next; return PS_OK;
        }
        case PS_OPT_QUEUE_GROUPS:
            if (value < 1) return PS_ERR_INVALID_ARG;
            ps->queue_groups = value; return PS_OK;
        case PS_OPT_LOG_UPDATES:
            if (value < 0) return PS_ERR_INVALID_ARG;
            ps->log_updates = value; return PS_OK;
        case PS_OPT_TIMING:
            if (value != 0 && value != 1) return PS_ERR_INVALID_ARG;
            ps->timing = static_cast<int>(value); return PS_OK;
        case PS_OPT_KERNEL:
            if (value < PS_KERNEL_AUTO || value > PS_KERNEL_BULK) return PS_ERR_INVALID_ARG;
            ps->kernel_choice = static_cast<int>(value); return PS_OK;
        case PS_OPT_BULK_TILE:
            if (value != 0 && (value < 256 || value > 8192 || (value & (value - 1)))) return PS_ERR_INVALID_ARG;
            ps->bulk_tile = static_cast<int>(value); return PS_OK;
        case PS_OPT_BULK_STAGES:
            if (value < 2 || value > softsync::kBulkMaxStages) return PS_ERR_INVALID_ARG;
            ps->bulk_stages = static_cast<int>(value); return PS_OK;
        case PS_OPT_BULK_WAIT_LIMIT:
            if (value < 16 || value > (int64_t{1} << 30)) return PS_ERR_INVALID_ARG;
            ps->bulk_wait_limit = static_cast<int>(value); return PS_OK;
        case PS_OPT_BULK_SELFTEST:
            if (value != 0 && value != 1) return PS_ERR_INVALID_ARG;
            ps->bulk_selftest = static_cast<int>(value); return PS_OK;
        case PS_OPT_PROTOCOL:
            if (value != PS_PROTOCOL_SOFTSYNC && value != PS_PROTOCOL_HARDSYNC) return PS_ERR_INVALID_ARG;
            if (value == PS_PROTOCOL_HARDSYNC && ps->split != 1) return PS_ERR_INVALID_ARG;
            if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
            ps->protocol = static_cast<int>(value); return PS_OK;
        case PS_OPT_OVERLAP_LAUNCH:
            if (value != 0 && value != 1) return PS_ERR_INVALID_ARG;
            ps->overlap_launch = static_cast<int>(value); return PS_OK;
        case PS_OPT_BLOCK_THREADS:
            if (value != 0 && value != 128 && value != 256 && value != 512) return PS_ERR_INVALID_ARG;
            ps->block_threads = static_cast<int>(value); return PS_OK;
        case PS_OPT_ZIGZAG:
            if (value != 0 && value != 1) return PS_ERR_INVALID_ARG;
            ps->zigzag = static_cast<int>(value); return PS_OK;
        default:
            return PS_ERR_INVALID_ARG;
        }
    } PS_CATCH_ALL
}

int ps_get_option(ps_t *ps, int key, int64_t *value)
{
    try {
        if (!is_live(ps) || !value) return PS_ERR_INVALID_ARG;
        switch (key) {
        case PS_OPT_GRAD_DTYPE: *value = ps->grad_dtype; return PS_OK;
        case PS_OPT_FUSE_T: *value = ps->fuse_t; return PS_OK;
        case PS_OPT_STREAM: *value = static_cast<int64_t>(reinterpret_cast<uintptr_t>(ps->stream)); return PS_OK;
        case PS_OPT_QUEUE_GROUPS: *value = ps->queue_groups; return PS_OK;
        case PS_OPT_LOG_UPDATES: *value = ps->log_updates; return PS_OK;
        case PS_OPT_TIMING: *value = ps->timing; return PS_OK;
        case PS_OPT_KERNEL: *value = ps->kernel_choice; return PS_OK;
        case PS_OPT_BLOCK_THREADS: *value = ps->block_threads; return PS_OK;
        case PS_OPT_OVERLAP_LAUNCH: *value = ps->overlap_launch; return PS_OK;
        case PS_OPT_PROTOCOL: *value = ps->protocol; return PS_OK;
        case PS_OPT_GROUP_SIZE: *value = ps->c; return PS_OK;
        case PS_OPT_LAST_KERNEL: *value = ps->last_kernel; return PS_OK;
        case PS_OPT_LAUNCHES_SCALAR: *value = ps->launches_by_kind[PS_KERNEL_SCALAR]; return PS_OK;
        case PS_OPT_LAUNCHES_VECTOR: *value = ps->launches_by_kind[PS_KERNEL_VECTOR]; return PS_OK;
        case PS_OPT_LAUNCHES_BULK: *value = ps->launches_by_kind[PS_KERNEL_BULK]; return PS_OK;
        case PS_OPT_BULK_TILE: *value = ps->bulk_tile; return PS_OK;
        case PS_OPT_BULK_STAGES: *value = ps->bulk_stages; return PS_OK;
        case PS_OPT_BULK_WAIT_LIMIT: *value = ps->bulk_wait_limit; return PS_OK;
        case PS_OPT_BULK_SELFTEST: *value = ps->bulk_selftest; return PS_OK;
        case PS_OPT_ZIGZAG: *value = ps->zigzag; return PS_OK;
        default: return PS_ERR_INVALID_ARG;
        }
    } PS_CATCH_ALL
}

int ps_set_alpha0(ps_t *ps, float alpha0)
{
    try {
        if (!is_live(ps) || !(alpha0 == alpha0)) return PS_ERR_INVALID_ARG;
        ps->alpha0 = alpha0;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_set_penalty_base(ps_t *ps, float rho)
{
    try {
        if (!is_live(ps) || !(rho > 0.0f) || rho > 1.0f) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
        ps->penalty_base = rho;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_set_layer_multipliers(ps_t *ps, int num_layers, const int64_t *bounds, const float *lr_mult, const float *wd_mult)
{
    try {
        if (!is_live(ps) || num_layers < 0 || num_layers > PS_MAX_LAYERS) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_INVALID_ARG;
        if (num_layers == 0) { ps->num_layers = 0; return PS_OK; }
        if (!bounds || !lr_mult || !wd_mult) return PS_ERR_INVALID_ARG;
        if (bounds[0] != 0 || bounds[num_layers] != ps->n) return PS_ERR_INVALID_ARG;
        for (int q = 0; q < num_layers; ++q) {
            if (bounds[q] > bounds[q + 1]) return PS_ERR_INVALID_ARG;
            if (!(lr_mult[q] == lr_mult[q]) || !(wd_mult[q] == wd_mult[q])) return PS_ERR_INVALID_ARG;
        }
        ps->num_layers = num_layers;
        for (int q = 0; q < num_layers; ++q) {
            ps->layer_end[q] = bounds[q + 1]; ps->layer_lr[q] = lr_mult[q]; ps->layer_wd[q] = wd_mult[q];
        }
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_apply_update(ps_t *ps)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        return apply_some(ps);
    } PS_CATCH_ALL
}

int ps_flush(ps_t *ps)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        int total = 0;
        while (!ps->ready.empty()) {
            const int r = apply_some(ps);
            if (r < 0) return r;
            total += r;
        }
        return total;
    } PS_CATCH_ALL
}

int ps_pull_weights(ps_t *ps, float *out_dev, int64_t *ts)
{
    try {
        if (!is_live(ps) || !ts) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (out_dev) {
            if (ps->n > 0 && (!ps->w || !ps->v)) return PS_ERR_NO_STATE;
            const int r = ps_flush(ps);                       // weights must belong to the returned timestamp
            if (r < 0) return r;
            if (ps->n) PS_CUDA(ps, cudaMemcpyAsync(out_dev, ps->w, static_cast<size_t>(ps->n) * sizeof(float),
                                                   cudaMemcpyDeviceToDevice, ps->stream));
        }
        *ts = ts_logical(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_pull_weights_bf16(ps_t *ps, void *out_dev, int64_t *ts)
{
    try {
        if (!is_live(ps) || !ts || !out_dev) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (!ps->mirror || (ps->n > 0 && (!ps->w || !ps->v))) return PS_ERR_NO_STATE;
        const int r = ps_flush(ps);
        if (r < 0) return r;
        if (ps->n) PS_CUDA(ps, cudaMemcpyAsync(out_dev, ps->mirror, static_cast<size_t>(ps->n) * 2,
                                               cudaMemcpyDeviceToDevice, ps->stream));
        *ts = ts_logical(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_pull_weights_host(ps_t *ps, float *out_host, int64_t *ts)
{
    try {
        if (!is_live(ps) || !ts || !out_host) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (!ps->w || !ps->v) return PS_ERR_NO_STATE;
        const int r = ps_flush(ps);
        if (r < 0) return r;
        if (ps->n) PS_CUDA(ps, cudaMemcpyAsync(out_host, ps->w, static_cast<size_t>(ps->n) * sizeof(float),
                                               cudaMemcpyDeviceToHost, ps->stream));
        PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
        *ts = ts_logical(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_pull_weights_host_async(ps_t *ps, float *out_host, int64_t *ts)
{
    try {
        if (!is_live(ps) || !ts || !out_host) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (!ps->w || !ps->v) return PS_ERR_NO_STATE;
        const int r = ps_flush(ps);
        if (r < 0) return r;
        if (!ps->copy_stream) {
            PS_CUDA(ps, cudaStreamCreateWithFlags(&ps->copy_stream, cudaStreamNonBlocking));
            PS_CUDA(ps, cudaEventCreateWithFlags(&ps->weights_ready, cudaEventDisableTiming));
            PS_CUDA(ps, cudaEventCreateWithFlags(&ps->weights_copied, cudaEventDisableTiming));
        }
        if (ps->n) {
            PS_CUDA(ps, cudaEventRecord(ps->weights_ready, ps->stream));
            PS_CUDA(ps, cudaStreamWaitEvent(ps->copy_stream, ps->weights_ready, 0));
            PS_CUDA(ps, cudaMemcpyAsync(out_host, ps->w, static_cast<size_t>(ps->n) * sizeof(float),
                                        cudaMemcpyDeviceToHost, ps->copy_stream));
            PS_CUDA(ps, cudaEventRecord(ps->weights_copied, ps->copy_stream));
            ps->copy_in_flight = true;
        }
        *ts = ts_logical(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_push_gradient(ps_t *ps, int learner, const void *grad_dev, int64_t ts)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        const int rc = check_push(ps, learner, grad_dev, ts);
        if (rc != PS_OK) return rc;
        if (reinterpret_cast<uintptr_t>(grad_dev) & (grad_elem_bytes(ps) - 1)) return PS_ERR_INVALID_ARG;
        return push_common(ps, learner, grad_dev, ts, -1);
    } PS_CATCH_ALL
}

int ps_push_gradient_host(ps_t *ps, int learner, const void *grad_host, int64_t ts)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        const int rc = check_push(ps, learner, grad_host, ts);
        if (rc != PS_OK) return rc;
        if (ps->n == 0) return push_common(ps, learner, nullptr, ts, -1);   // nothing to copy, nothing to stage
        if (!ps->staging) return PS_ERR_NO_STATE;
        if (ps->free_slots.empty()) return PS_ERR_QUEUE_FULL;
        const int slot = ps->free_slots.back();
        char *dst = ps->staging + static_cast<int64_t>(slot) * ps->slot_bytes;
        const size_t bytes = static_cast<size_t>(ps->n) * grad_elem_bytes(ps);
        if (bytes) PS_CUDA(ps, cudaMemcpyAsync(dst, grad_host, bytes, cudaMemcpyHostToDevice, ps->stream));
        ps->free_slots.pop_back();
        return push_common(ps, learner, dst, ts, slot);
    } PS_CATCH_ALL
}

int ps_acquire_slot(ps_t *ps, void **slot_dev, int *slot_id)
{
    try {
        if (!is_live(ps) || !slot_dev || !slot_id) return PS_ERR_INVALID_ARG;
        if (!ps->staging) return PS_ERR_NO_STATE;
        if (ps->free_slots.empty()) return PS_ERR_QUEUE_FULL;
        const int slot = ps->free_slots.back();
        ps->free_slots.pop_back();
        ps->slot_lent[slot] = 1;
        *slot_id = slot;
        *slot_dev = ps->staging + static_cast<int64_t>(slot) * ps->slot_bytes;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_release_slot(ps_t *ps, int slot_id)
{
    try {
        if (!is_live(ps) || slot_id < 0 || slot_id >= ps->num_slots || !ps->slot_lent[slot_id]) return PS_ERR_INVALID_ARG;
        ps->slot_lent[slot_id] = 0;
        ps->free_slots.push_back(slot_id);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_push_slot(ps_t *ps, int learner, int slot_id, int64_t ts)
{
    try {
        if (!is_live(ps) || slot_id < 0 || slot_id >= ps->num_slots || !ps->slot_lent[slot_id]) return PS_ERR_INVALID_ARG;
        const void *grad = ps->staging + static_cast<int64_t>(slot_id) * ps->slot_bytes;
        const int rc = check_push(ps, learner, grad, ts);
        if (rc != PS_OK) return rc;                       // the learner keeps the slot and may try again
        ps->slot_lent[slot_id] = 0;
        return push_common(ps, learner, grad, ts, slot_id, true);
    } PS_CATCH_ALL
}

int ps_slot_wait(ps_t *ps, int slot_id, void *stream)
{
    try {
        if (!is_live(ps) || slot_id < 0 || slot_id >= ps->num_slots || !ps->slot_lent[slot_id]) return PS_ERR_INVALID_ARG;
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        if (st == ps->stream || !ps->slot_has_consumer[slot_id]) return PS_OK;   // stream order covers it / never read yet
        DeviceGuard on_device(ps);
        PS_CUDA(ps, cudaStreamWaitEvent(st, ps->slot_consumed[slot_id], 0));
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_slot_written(ps_t *ps, int slot_id, void *stream)
{
    try {
        if (!is_live(ps) || slot_id < 0 || slot_id >= ps->num_slots || !ps->slot_lent[slot_id]) return PS_ERR_INVALID_ARG;
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        if (st == ps->stream) return PS_OK;
        DeviceGuard on_device(ps);
        if (!ps->slot_filled[slot_id])
            PS_CUDA(ps, cudaEventCreateWithFlags(&ps->slot_filled[slot_id], cudaEventDisableTiming));
        PS_CUDA(ps, cudaEventRecord(ps->slot_filled[slot_id], st));
        PS_CUDA(ps, cudaStreamWaitEvent(ps->stream, ps->slot_filled[slot_id], 0));
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_synchronize(ps_t *ps)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
        if (ps->copy_stream) PS_CUDA(ps, cudaStreamSynchronize(ps->copy_stream));
        if (ps->bulk_status && ps->bulk_status->code != 0) return PS_ERR_DEVICE_WAIT;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_kernel_status(ps_t *ps, int *code, int *block, int64_t *tile, int *stage)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        if (ps->device >= 0) PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
        const BulkStatus st = ps->bulk_status ? *ps->bulk_status : BulkStatus{0, 0, 0, 0};
        if (code) *code = st.code;
        if (block) *block = st.block;
        if (tile) *tile = st.tile;
        if (stage) *stage = st.stage;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_get_update_log(ps_t *ps, int64_t first_update, int64_t count, ps_log_entry *out_host)
{
    try {
        if (!is_live(ps) || count < 0 || (count > 0 && !out_host)) return PS_ERR_INVALID_ARG;
        const int64_t held = static_cast<int64_t>(ps->log.size()) / ps->c;
        if (first_update < ps->log_first_update || first_update + count > ps->log_first_update + held)
            return PS_ERR_LOG_EVICTED;
        const int64_t off = (first_update - ps->log_first_update) * ps->c;
        std::copy(ps->log.begin() + off, ps->log.begin() + off + count * ps->c, out_host);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_peek_state(ps_t *ps, const float **w_dev, const float **v_dev, int64_t *ts_applied, int64_t *ts_log)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        if (w_dev) *w_dev = ps->w;
        if (v_dev) *v_dev = ps->v;
        if (ts_applied) *ts_applied = ps->ts_applied;
        if (ts_log) *ts_log = ts_logical(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

namespace {
constexpr int64_t kStateMagic = 0x5053534F46545359LL;   // "PSSOFTSY"
constexpr int64_t kStateVersion = 1;
constexpr int64_t kStateHeader = 8;
}  // namespace

int ps_export_state(ps_t *ps, int64_t *out_host, int64_t capacity_words)
{
    try {
        if (!is_live(ps) || !out_host) return PS_ERR_INVALID_ARG;
        const int64_t words = kStateHeader + ps->lambda;
        if (capacity_words < words) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_NOT_READY;   // borrowed gradients cannot be saved
        uint32_t alpha_bits;
        static_assert(sizeof alpha_bits == sizeof ps->alpha0, "fp32 rate");
        std::memcpy(&alpha_bits, &ps->alpha0, sizeof alpha_bits);
        out_host[0] = kStateMagic; out_host[1] = kStateVersion;
        out_host[2] = ps->n; out_host[3] = ps->lambda; out_host[4] = ps->split;
        out_host[5] = ps->ts_applied; out_host[6] = static_cast<int64_t>(alpha_bits); out_host[7] = ps->launches;
        for (int l = 0; l < ps->lambda; ++l) out_host[kStateHeader + l] = ps->push_count[l];
        return static_cast<int>(words);
    } PS_CATCH_ALL
}

int ps_import_state(ps_t *ps, const int64_t *in_host, int64_t words)
{
    try {
        if (!is_live(ps) || !in_host || words < kStateHeader) return PS_ERR_INVALID_ARG;
        if (in_host[0] != kStateMagic || in_host[1] != kStateVersion) return PS_ERR_INVALID_ARG;
        if (in_host[2] != ps->n || in_host[3] != ps->lambda || in_host[4] != ps->split) return PS_ERR_INVALID_ARG;
        if (words != kStateHeader + ps->lambda || in_host[5] < 0 || in_host[7] < 0) return PS_ERR_INVALID_ARG;
        for (int l = 0; l < ps->lambda; ++l) if (in_host[kStateHeader + l] < 0) return PS_ERR_INVALID_ARG;
        if (!ps->ready.empty() || !ps->filling.empty()) return PS_ERR_NOT_READY;
        const uint32_t alpha_bits = static_cast<uint32_t>(in_host[6]);
        float alpha0;
        std::memcpy(&alpha0, &alpha_bits, sizeof alpha0);
        if (!(alpha0 == alpha0)) return PS_ERR_INVALID_ARG;
        ps->alpha0 = alpha0;
        ps->ts_applied = in_host[5];
        ps->launches = in_host[7];
        for (int l = 0; l < ps->lambda; ++l) ps->push_count[l] = in_host[kStateHeader + l];
        ps->log.clear();
        ps->log_first_update = ps->ts_applied;
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_kernel_time(ps_t *ps, double *total_ms, int64_t *launches)
{
    try {
        if (!is_live(ps)) return PS_ERR_INVALID_ARG;
        DeviceGuard on_device(ps);
        PS_CUDA(ps, cudaStreamSynchronize(ps->stream));
        double sum = 0.0;
        for (const auto &tl : ps->timed) {
            float ms = 0.f;
            PS_CUDA(ps, cudaEventElapsedTime(&ms, tl.start, tl.stop));
            sum += ms;
        }
        if (total_ms) *total_ms = sum;
        if (launches) *launches = static_cast<int64_t>(ps->timed.size());
        release_events(ps);
        return PS_OK;
    } PS_CATCH_ALL
}

int ps_last_cuda_error(ps_t *ps)
{
    return is_live(ps) ? ps->last_cuda_error : 0;
}

const char *ps_status_string(int status)
{
    switch (status) {
    case PS_OK: return "ok";
    case PS_READY: return "ready: a group of c gradients is complete";
    case PS_ERR_INVALID_ARG: return "invalid argument";
    case PS_ERR_BAD_LEARNER: return "learner id out of range";
    case PS_ERR_BAD_TIMESTAMP: return "gradient timestamp negative or ahead of the server";
    case PS_ERR_NOT_READY: return "no complete group is pending";
    case PS_ERR_QUEUE_FULL: return "too many unapplied groups or no free staging slot";
    case PS_ERR_CUDA: return "CUDA call failed";
    case PS_ERR_NOMEM: return "host allocation failed";
    case PS_ERR_NO_STATE: return "weights, momentum or staging slots not bound";
    case PS_ERR_LOG_EVICTED: return "log range not held";
    case PS_ERR_BARRIER: return "hardsync: learner already contributed to this round";
    case PS_ERR_DEVICE_WAIT: return "an update kernel gave up on a bounded wait; re-initialise the weights";
    case PS_ERR_STATIC_LIMIT: return "more blocks or gradients than the static status area of ps_fused_update_static holds";
    default: return status > 1 ? "updates applied" : "unknown status";
    }
}

}  // extern "C"

// =====================================================================================
// ps_fused_update_static: one update by the bulk-copy kernel for callers that must not
// allocate.  The kernel's status records live in static device memory instead of memory
// obtained at run time.
// =====================================================================================
namespace {

// One record per block of the largest grid the entry point accepts.  In host code this name is only a
// stand-in for the symbol: the address a kernel can use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) BulkStatus g_static_records[PS_STATIC_MAX_BLOCKS];

constexpr int kStaticMaxDevices = 64;
constexpr int kStaticStages = 2;
constexpr int kStaticWaitLimit = 1 << 20;

struct StaticSetup {
    bool done = false;
    BulkStatus *records = nullptr;     // device address of g_static_records on this device
    int sm_count = 0;
};
StaticSetup g_static_setup[kStaticMaxDevices];
std::mutex g_static_mutex;

using StaticParams = LaunchParams<kHead, 1>;

template <typename GT>
auto static_kernel() { return softsync::softsync_update_bulk_kernel<GT, false, kHead, 1, true>; }

// First use on a device: the device address of the record array and the kernel's shared-memory opt-in.
cudaError_t static_setup(int device, StaticSetup **out)
{
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticSetup &st = g_static_setup[device];
    if (!st.done) {
        BulkStatus *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&ptr), g_static_records);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(static_kernel<GradFp32>(), cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(static_kernel<GradBf16>(), cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return e;
        st.records = ptr;
        st.done = true;
    }
    *out = &st;
    return cudaSuccess;
}

}  // namespace

extern "C" int ps_fused_update_static(float *w_dev, float *v_dev, int64_t num_params,
                                      const void *const *grads_dev, const float *scales_host, int c,
                                      float decay, float momentum, int grad_dtype,
                                      int blocks, void *stream, int *blocks_gave_up)
{
  try {
    if (num_params < 0 || c < 1 || blocks < 0) return PS_ERR_INVALID_ARG;
    if (grad_dtype != PS_GRAD_FP32 && grad_dtype != PS_GRAD_BF16) return PS_ERR_INVALID_ARG;
    if (c > PS_STATIC_MAX_GRADS || blocks > PS_STATIC_MAX_BLOCKS) return PS_ERR_STATIC_LIMIT;
    if (!grads_dev || !scales_host) return PS_ERR_INVALID_ARG;
    if (blocks_gave_up) *blocks_gave_up = 0;
    if (num_params == 0) return PS_OK;
    if (!w_dev || !v_dev || w_dev == v_dev || !aligned16(w_dev) || !aligned16(v_dev)) return PS_ERR_INVALID_ARG;
    for (int l = 0; l < c; ++l)
        if (!grads_dev[l] || !aligned16(grads_dev[l])) return PS_ERR_INVALID_ARG;

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kStaticMaxDevices) return PS_ERR_CUDA;
    StaticSetup *setup = nullptr;
    if (static_setup(device, &setup) != cudaSuccess) return PS_ERR_CUDA;

    StaticParams p;
    p.w = w_dev; p.v = v_dev; p.n = num_params;
    p.momentum = make_float2(momentum, momentum); p.T = 1; p.c = c;
    p.overlap = 0; p.reverse = 0; p.mirror = nullptr; p.nrep = 0;
    p.layers.count = 0;
    p.d[0] = make_float2(decay, decay);
    for (int l = 0; l < c; ++l) { p.s[l] = make_float2(scales_host[l], scales_host[l]); p.g[l] = grads_dev[l]; }

    // the launch shape of the PS_KERNEL_BULK default
    const int gb = grad_dtype == PS_GRAD_BF16 ? 2 : 4;
    const BulkShape sh = bulk_shape(c, gb, kStaticStages, 0, 0);
    const int tile = sh.tile;
    const size_t smem = sh.smem;

    BulkPlan plan;
    plan.tile_elems = tile;
    plan.ntiles = num_params / tile;
    plan.stages = kStaticStages;
    plan.wait_limit = kStaticWaitLimit;
    plan.selftest = 0;
    plan.status = setup->records;
    long long grid = std::max<long long>(1, std::min<long long>(plan.ntiles, static_cast<long long>(sh.blocks_per_sm) * setup->sm_count));
    if (blocks > 0) grid = std::min<long long>(grid, blocks);
    if (grid > PS_STATIC_MAX_BLOCKS) return PS_ERR_STATIC_LIMIT;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array still holds what the previous call left: clear the records this grid will use
    if (cudaMemsetAsync(setup->records, 0, static_cast<size_t>(grid) * sizeof(BulkStatus), st) != cudaSuccess) return PS_ERR_CUDA;
    const dim3 g(static_cast<unsigned>(grid)), b(static_cast<unsigned>(sh.threads));
    if (grad_dtype == PS_GRAD_BF16)
        softsync::softsync_update_bulk_kernel<GradBf16, false, kHead, 1, true><<<g, b, smem, st>>>(p, plan);
    else
        softsync::softsync_update_bulk_kernel<GradFp32, false, kHead, 1, true><<<g, b, smem, st>>>(p, plan);
    if (cudaGetLastError() != cudaSuccess) return PS_ERR_CUDA;

    if (blocks_gave_up) {
        BulkStatus seen[PS_STATIC_MAX_BLOCKS];
        if (cudaStreamSynchronize(st) != cudaSuccess) return PS_ERR_CUDA;
        if (cudaMemcpy(seen, setup->records, static_cast<size_t>(grid) * sizeof(BulkStatus), cudaMemcpyDeviceToHost) != cudaSuccess)
            return PS_ERR_CUDA;
        int gave_up = 0;
        for (long long k = 0; k < grid; ++k) gave_up += seen[k].code != 0;
        *blocks_gave_up = gave_up;
    }
    return PS_OK;
  } PS_CATCH_ALL
}
