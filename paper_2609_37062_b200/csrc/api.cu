// Host side of the C ABI: plan objects, argument checks, kernel selection and
// launches.  No device memory is allocated in run/combine; the plan owns one
// small device buffer (work list, per-sequence split table, tickets, status).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstddef>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "append.cuh"
#include "combine.cuh"
#include "common.cuh"
#include "decode_attn.h"
#include "kernel_mma.cuh"
#include "kernel_umma.cuh"
#include "kernel_simt.cuh"
#include "planner.h"

using namespace da;

#define DA_CUDA_TRY(expr)                         \
    do {                                          \
        cudaError_t err__ = (expr);               \
        if (err__ != cudaSuccess) {               \
            (void)cudaGetLastError();             \
            return DA_ERR_CUDA;                   \
        }                                         \
    } while (0)

struct decode_attn_plan {
    decode_attn_shape_t shape;
    decode_attn_policy_t policy;
    Layout layout;
    std::vector<int32_t> seq_lens;
    int device = -1;
    int sm_count = 0;
    int ctas_per_sm = 0;
    int kernel = DA_KERNEL_SIMT;
    int group = 1;
    int block_threads = 0;
    int dyn_smem = 0;
    float scale = 0.f;
    int64_t max_units = 0;   // capacity of the device work list
    int64_t max_batch = 0;
    int64_t max_slots = 0;   // what the workspace is sized for
    int64_t grid = 0;        // blocks launched by run: work_grid attending blocks (+ merge blocks when fused)
    int64_t work_grid = 0;
    size_t workspace_bytes = 0;
    // device buffer (views into the cached allocation the plan holds)
    char* dev = nullptr;
    char* pinned = nullptr;
    size_t upload_bytes = 0;
    size_t off_units = 0, off_seq_info = 0, off_block_begin = 0, off_unit_rank = 0, off_status = 0, off_tickets = 0, off_queue = 0,
           total_bytes = 0;
    int max_bins = 0;        // > 0: the units are packed into per-block ranges (persistent tensor-core kernel)
    cudaStream_t stream = nullptr;
    cudaEvent_t upload_done = nullptr;  // last refresh of the device work list
    cudaEvent_t launch_done = nullptr;  // behind the plan's last launch on a caller's stream (not while capturing)
    mutable bool upload_pending = false;   // the first upload may still be in flight on the plan's own stream
    void* buffers = nullptr;            // PlanBuffers*, returned to the cache on destroy
};

#ifdef DA_TRACE
static unsigned long long* g_trace_buffer = nullptr;
#endif
namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// page_size is a power of two (validate_shape).
int log2_of(int x)
{
    int r = 0;
    while ((1 << (r + 1)) <= x) ++r;
    return r;
}

int out_kind_of(int out_dtype) { return out_dtype == DA_DTYPE_BF16 ? 1 : out_dtype == DA_DTYPE_FP16 ? 2 : 0; }

// Device buffer, pinned mirror, stream and event of a plan.  Creating these
// costs far more than planning a step, so destroyed plans park theirs here
// and the next plan of a similar size picks them up.
struct PlanBuffers {
    int device = -1;
    char* dev = nullptr;
    char* pinned = nullptr;
    size_t dev_bytes = 0, pinned_bytes = 0;
    cudaStream_t stream = nullptr;
    cudaEvent_t event = nullptr;        // upload of the work list
    cudaEvent_t launched = nullptr;     // behind the last kernel that reads the device buffer
};

void free_buffers(PlanBuffers& b)
{
    if (b.stream) {
        cudaStreamSynchronize(b.stream);
        cudaStreamDestroy(b.stream);
    }
    if (b.launched) {
        cudaEventSynchronize(b.launched);     // kernels of the plan that held these buffers may still run
        cudaEventDestroy(b.launched);
    }
    if (b.event) cudaEventDestroy(b.event);
    if (b.dev) cudaFree(b.dev);
    if (b.pinned) cudaFreeHost(b.pinned);
    (void)cudaGetLastError();
    b = PlanBuffers();
}

struct BufferCache {
    std::mutex mu;
    std::vector<PlanBuffers> free_list;
    static constexpr size_t kMaxParked = 8;
} g_buffers;

size_t round_pow2(size_t x)
{
    size_t r = 4096;
    while (r < x) r <<= 1;
    return r;
}

int acquire_buffers(int device, size_t dev_bytes, size_t pinned_bytes, PlanBuffers* out)
{
    {
        std::lock_guard<std::mutex> lock(g_buffers.mu);
        for (size_t i = 0; i < g_buffers.free_list.size(); ++i) {
            PlanBuffers& b = g_buffers.free_list[i];
            if (b.device == device && b.dev_bytes >= dev_bytes && b.pinned_bytes >= pinned_bytes) {
                *out = b;
                g_buffers.free_list.erase(g_buffers.free_list.begin() + i);
                return DA_OK;
            }
        }
    }
    PlanBuffers b;
    b.device = device;
    b.dev_bytes = round_pow2(dev_bytes);
    b.pinned_bytes = round_pow2(pinned_bytes);
    if (cudaStreamCreateWithFlags(&b.stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&b.event, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&b.launched, cudaEventDisableTiming) != cudaSuccess ||
        cudaMalloc(&b.dev, b.dev_bytes) != cudaSuccess || cudaMallocHost(&b.pinned, b.pinned_bytes) != cudaSuccess) {
        (void)cudaGetLastError();
        free_buffers(b);
        return DA_ERR_CUDA;
    }
    *out = b;
    return DA_OK;
}

// Parks the buffers of a destroyed plan without waiting for the device: kernels of that plan may
// still be running on the caller's stream (a step is plan / run / combine / destroy with no
// synchronisation in between).  Whoever takes the buffers next orders its upload behind `launched`
// (see decode_attn_plan) and waits for `event` on the host before it rewrites the pinned mirror.
void release_buffers(PlanBuffers& b)
{
    if (!b.dev) return;
    {
        std::lock_guard<std::mutex> lock(g_buffers.mu);
        if (g_buffers.free_list.size() < BufferCache::kMaxParked) {
            g_buffers.free_list.push_back(b);
            b = PlanBuffers();
            return;
        }
    }
    free_buffers(b);
}

typedef void (*simt_kernel_t)(const KernelParams);

template <int D>
simt_kernel_t simt_for_group(int G)
{
    switch (G) {
        case 1: return decode_attn_simt_kernel<D, 1>;
        case 2: return decode_attn_simt_kernel<D, 2>;
        case 3: return decode_attn_simt_kernel<D, 3>;
        case 4: return decode_attn_simt_kernel<D, 4>;
        case 5: return decode_attn_simt_kernel<D, 5>;
        case 6: return decode_attn_simt_kernel<D, 6>;
        case 7: return decode_attn_simt_kernel<D, 7>;
        case 8: return decode_attn_simt_kernel<D, 8>;
        default: return nullptr;
    }
}

simt_kernel_t simt_kernel_for(int D, int G)
{
    return D == 64 ? simt_for_group<64>(G) : D == 128 ? simt_for_group<128>(G) : nullptr;
}

// Launch with a programmatic dependency on the kernel before (see pdl_wait_primary).
int simt_launch(simt_kernel_t fn, const KernelParams& kp, unsigned grid, cudaStream_t stream)
{
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kSimtThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, fn, kp) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

int pick_kernel(const decode_attn_shape_t& s, const decode_attn_policy_t& p)
{
    if (p.kernel != DA_KERNEL_AUTO) return p.kernel;
    const int G = s.num_q_heads / s.num_kv_heads;
    if (p.shared_prefix_tokens > 0 && umma_supports(s.head_dim, G)) return DA_KERNEL_UMMA_PREFIX;
    // The TMA-fed kernel wins at every group size, group 1 included (no reuse for the tensor core
    // there, but the stream is what counts: 7.1 against 5.1 TB/s on 1 GB of MHA cache).
    return mma_supports(s.head_dim, G) ? DA_KERNEL_MMA_TMA : DA_KERNEL_SIMT;
}

// Resident blocks per SM of the kernel a plan will launch (the uncached query; it also opts the
// kernel in to its dynamic shared memory).
int query_occupancy_uncached(int kernel, int D, int G, int* block_threads, int* dyn_smem, bool prefix)
{
    int n = 0;
    if (kernel == DA_KERNEL_SIMT) {
        simt_kernel_t fn = simt_kernel_for(D, G);
        if (!fn) return -1;
        *block_threads = kSimtThreads;
        *dyn_smem = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, fn, kSimtThreads, 0) != cudaSuccess) {
            (void)cudaGetLastError();
            return -1;
        }
        return n;
    }
    return mma_query_occupancy(D, G, block_threads, dyn_smem, prefix);
}

// Plans are made every decode step: the answers that depend only on (device, kernel variant) are
// kept after the first query.
struct OccEntry {
    int device, kernel, D, G, prefix, occ, block_threads, dyn_smem;
};
std::mutex g_occ_mu;
std::vector<OccEntry> g_occ;
std::vector<std::pair<int, int>> g_sm_counts;   // (device, multiprocessors)

int query_occupancy(int kernel, int D, int G, int* block_threads, int* dyn_smem, bool prefix = false)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    {
        std::lock_guard<std::mutex> lock(g_occ_mu);
        for (const OccEntry& e : g_occ)
            if (e.device == dev && e.kernel == kernel && e.D == D && e.G == G && e.prefix == (int)prefix) {
                *block_threads = e.block_threads;
                *dyn_smem = e.dyn_smem;
                return e.occ;
            }
    }
    const int occ = query_occupancy_uncached(kernel, D, G, block_threads, dyn_smem, prefix);
    if (occ > 0) {
        std::lock_guard<std::mutex> lock(g_occ_mu);
        g_occ.push_back({dev, kernel, D, G, (int)prefix, occ, *block_threads, *dyn_smem});
    }
    return occ;
}

int device_sm_count(int dev, int* out)
{
    {
        std::lock_guard<std::mutex> lock(g_occ_mu);
        for (const auto& e : g_sm_counts)
            if (e.first == dev) {
                *out = e.second;
                return DA_OK;
            }
    }
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_occ_mu);
    g_sm_counts.push_back({dev, n});
    *out = n;
    return DA_OK;
}

// Launches with a RUN mask hand the binned units out in cost order (see the kernel's queue): the
// plan uploads their positions by rank.
bool ranked_fits(const decode_attn_plan_t* pl)
{
    return pl->max_bins > 0 && !pl->layout.rank_pos.empty();
}

void fill_host_mirror(decode_attn_plan_t* pl)
{
    DevHeader* hdr = reinterpret_cast<DevHeader*>(pl->pinned);
    hdr->n_units = (int32_t)pl->layout.units.size();
    hdr->batch = pl->shape.batch;
    hdr->n_ranked = ranked_fits(pl) ? (int32_t)pl->layout.rank_pos.size() : 0;
    hdr->first_binned = pl->layout.n_front_units;
    std::memcpy(pl->pinned + pl->off_units, pl->layout.units.data(),
                pl->layout.units.size() * sizeof(decode_attn_unit_t));
    SeqInfo* si = reinterpret_cast<SeqInfo*>(pl->pinned + pl->off_seq_info);
    for (int b = 0; b < pl->shape.batch; ++b) {
        si[b].slot_base = pl->layout.slot_base[b];
        si[b].n_splits = pl->layout.splits[b];
        si[b].seq_len = pl->seq_lens[b];
        si[b].pad = 0;
    }
    if (pl->max_bins > 0) {
        // one range per launched block; blocks beyond the bins in use get an empty range
        int32_t* bb = reinterpret_cast<int32_t*>(pl->pinned + pl->off_block_begin);
        const std::vector<int32_t>& src = pl->layout.block_begin;
        const int32_t end = (int32_t)pl->layout.units.size();
        for (int64_t i = 0; i <= pl->grid; ++i) bb[i] = i < (int64_t)src.size() ? src[i] : end;
        // every binned unit by cost rank: where it sits in the work list and whose row it is
        if (ranked_fits(pl)) {
            int2* ur = reinterpret_cast<int2*>(pl->pinned + pl->off_unit_rank);
            for (size_t j = 0; j < pl->layout.rank_pos.size(); ++j) {
                const int32_t pos = pl->layout.rank_pos[j];
                const decode_attn_unit_t& u = pl->layout.units[pos];
                ur[j] = make_int2(pos, (u.kv_head >> 16) ? -1 : u.seq);
            }
        }
    }
}

KernelParams make_params(const decode_attn_plan_t* pl, const decode_attn_run_args_t& a)
{
    KernelParams kp;
    std::memset(&kp, 0, sizeof kp);
    const decode_attn_shape_t& s = pl->shape;
    kp.q = static_cast<const __nv_bfloat16*>(a.q);
    kp.k = static_cast<const __nv_bfloat16*>(a.k_cache);
    kp.v = static_cast<const __nv_bfloat16*>(a.v_cache);
    kp.block_table = a.block_table;
    kp.seq_lens = a.seq_lens;
    kp.run_mask = a.run_mask;
    kp.new_k = static_cast<const __nv_bfloat16*>(a.new_k);
    kp.new_v = static_cast<const __nv_bfloat16*>(a.new_v);
    kp.out = a.out;
    kp.lse = a.lse;
    kp.ws = static_cast<float*>(a.workspace);
    kp.header = reinterpret_cast<const DevHeader*>(pl->dev);
    kp.units = reinterpret_cast<const decode_attn_unit_t*>(pl->dev + pl->off_units);
    kp.seq_info = reinterpret_cast<const SeqInfo*>(pl->dev + pl->off_seq_info);
    kp.block_begin = pl->max_bins > 0 ? reinterpret_cast<const int32_t*>(pl->dev + pl->off_block_begin) : nullptr;
    kp.unit_rank = reinterpret_cast<const int2*>(pl->dev + pl->off_unit_rank);
    kp.queue = pl->max_bins > 0 ? reinterpret_cast<int32_t*>(pl->dev + pl->off_queue) : nullptr;
    kp.n_ranked = ranked_fits(pl) ? (int32_t)pl->layout.rank_pos.size() : 0;
    kp.first_binned = pl->layout.n_front_units;
    kp.may_rank = pl->max_bins > 0 && pl->policy.capacity_batch > 0;
    kp.tickets = reinterpret_cast<int32_t*>(pl->dev + pl->off_tickets);
    kp.ticket_stride = (int32_t)(pl->max_batch * s.num_kv_heads);
    kp.batch = s.batch;
    kp.n_work_blocks = (int32_t)pl->work_grid;
    kp.status = reinterpret_cast<int32_t*>(pl->dev + pl->off_status);
    kp.k_stride_page = s.k_stride_page; kp.k_stride_token = s.k_stride_token; kp.k_stride_head = s.k_stride_head;
    kp.v_stride_page = s.v_stride_page; kp.v_stride_token = s.v_stride_token; kp.v_stride_head = s.v_stride_head;
    kp.num_pages = s.num_pages;
    kp.num_q_heads = s.num_q_heads;
    kp.num_kv_heads = s.num_kv_heads;
    kp.max_pages_per_seq = s.max_pages_per_seq;
    kp.scale_log2 = pl->scale * kLog2e;
    kp.out_kind = out_kind_of(s.out_dtype);
    kp.in_f16 = s.kv_dtype == DA_DTYPE_FP16;
    kp.tile_shift = log2_of(s.page_size) - 4;
    kp.fused = pl->policy.fuse_combine;
    kp.grid_exit = pl->policy.capacity_batch > 0;
    kp.n_units = (int32_t)pl->layout.units.size();
    kp.wait_limit = kWaitLimitCycles;
    // The tensor-core kernel asks the first pages of every block into L2 ahead of its dependency
    // wait.  Seven pages, just short of two stages' worth, when a block has a single unit (the opening
    // burst is then a visible share of the step: 24.8 us without hints, 23.9 / 23.6 / 23.2 / 23.2 /
    // 23.4 with 2 / 4 / 6 / 7 / 8 pages on one 32k sequence, more pages slower again), one stage's
    // worth otherwise (short_chat 20.0 -> 19.1 us).
    if (pl->kernel != DA_KERNEL_SIMT) {
        const bool single = pl->policy.capacity_batch == 0 &&
                            (int64_t)pl->layout.units.size() - pl->layout.n_front_units <= pl->work_grid;
        kp.hint_first_pages = single ? 7 : 4;
    }
#ifdef DA_TRACE
    kp.trace = g_trace_buffer;
#endif
    return kp;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bool stream_is_capturing(cudaStream_t stream)
{
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &st) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    return st != cudaStreamCaptureStatusNone;
}

// A plan's work list is uploaded on the plan's own stream without waiting for it.  Every launch
// that reads the device buffer is ordered behind that upload: a device-side wait on the caller's
// stream while the copy may still be in flight (a host-side one while that stream is being
// captured, so that no outside event enters the graph), nothing once it is known to be complete.
int order_behind_upload(const decode_attn_plan_t* pl, cudaStream_t stream)
{
    if (!pl->upload_pending) return DA_OK;
    const cudaError_t q = cudaEventQuery(pl->upload_done);
    if (q == cudaSuccess) {
        pl->upload_pending = false;
        return DA_OK;
    }
    (void)cudaGetLastError();
    if (q != cudaErrorNotReady) return DA_ERR_CUDA;
    if (stream_is_capturing(stream)) {
        DA_CUDA_TRY(cudaEventSynchronize(pl->upload_done));
        pl->upload_pending = false;
        return DA_OK;
    }
    DA_CUDA_TRY(cudaStreamWaitEvent(stream, pl->upload_done, 0));
    return DA_OK;
}

// Marks the end of the plan's launches on a caller's stream, so that the plan's device buffer is
// not handed to another plan's upload while they run (see release_buffers).  Launches that are
// being captured into a graph run later, at replay: a plan must outlive the replays of a graph
// that holds its launches, as the header says.
void mark_launched(const decode_attn_plan_t* pl, cudaStream_t stream)
{
    if (pl->launch_done == nullptr || stream_is_capturing(stream)) return;
    if (cudaEventRecord(pl->launch_done, stream) != cudaSuccess) (void)cudaGetLastError();
}

// marks the plan's launch on scope exit (for the entry points that return the launch's status)
struct mma_launch_guard {
    const decode_attn_plan_t* pl;
    cudaStream_t stream;
    ~mma_launch_guard() { mark_launched(pl, stream); }
};

}  // namespace

extern "C" {

int decode_attn_plan(const decode_attn_shape_t* shape, const decode_attn_policy_t* policy,
                     const int32_t* seq_lens_host, decode_attn_plan_t** plan_out, size_t* workspace_bytes_out)
{
    if (!shape || !policy || !plan_out) return DA_ERR_INVALID_ARG;
    if (shape->batch > 0 && !seq_lens_host) return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    rc = validate_policy(*shape, *policy);
    if (rc != DA_OK) return rc;

    decode_attn_plan_t* pl = new (std::nothrow) decode_attn_plan_t();
    if (!pl) return DA_ERR_INVALID_ARG;
    struct Guard {
        decode_attn_plan_t* p;
        ~Guard() { if (p) decode_attn_plan_destroy(p); }
    } guard{pl};

    pl->shape = *shape;
    pl->policy = *policy;
    pl->group = shape->num_q_heads / shape->num_kv_heads;
    pl->scale = shape->sm_scale > 0.f ? shape->sm_scale : 1.0f / sqrtf((float)shape->head_dim);
    pl->kernel = pick_kernel(*shape, *policy);
    if (pl->kernel != DA_KERNEL_SIMT && !mma_supports(shape->head_dim, pl->group)) return DA_ERR_UNSUPPORTED;
    if (pl->kernel == DA_KERNEL_SIMT && !simt_kernel_for(shape->head_dim, pl->group)) return DA_ERR_UNSUPPORTED;
    const bool umma = pl->kernel == DA_KERNEL_UMMA_PREFIX;
    if (umma && (!umma_supports(shape->head_dim, pl->group) || policy->shared_prefix_tokens <= 0)) return DA_ERR_UNSUPPORTED;
    pl->policy.kernel = pl->kernel;        // the planner cuts the prefix for the kernel that will run it

    DA_CUDA_TRY(cudaGetDevice(&pl->device));
    if (policy->sm_count > 0) {
        pl->sm_count = policy->sm_count;
    } else {
        rc = device_sm_count(pl->device, &pl->sm_count);
        if (rc != DA_OK) return rc;
    }
    const bool prefix = policy->shared_prefix_tokens > 0;
    if (prefix && pl->kernel == DA_KERNEL_SIMT) return DA_ERR_UNSUPPORTED;
    // what follows a tcgen05 prefix runs on the ordinary tensor-core kernel
    int occ = query_occupancy(DA_KERNEL_MMA_TMA == pl->kernel || umma ? DA_KERNEL_MMA_TMA : pl->kernel, shape->head_dim,
                              pl->group, &pl->block_threads, &pl->dyn_smem, prefix && !umma);
    if (occ <= 0) return DA_ERR_CUDA;
    pl->ctas_per_sm = policy->ctas_per_sm > 0 ? policy->ctas_per_sm : occ;

    pl->seq_lens.assign(seq_lens_host, seq_lens_host + shape->batch);
    // The tensor-core kernel walks the work list with a fixed set of resident blocks.
    if (pl->kernel != DA_KERNEL_SIMT) pl->max_bins = pl->sm_count * pl->ctas_per_sm;
    rc = make_layout(*shape, pl->policy, pl->seq_lens.data(), pl->sm_count, pl->ctas_per_sm, pl->layout, pl->max_bins);
    if (rc != DA_OK) return rc;

    if (policy->capacity_batch > 0) {
        pl->max_batch = policy->capacity_batch;
        pl->max_slots = capacity_slots(*shape, *policy);
        pl->max_units = (pl->max_slots + pl->max_batch) * shape->num_kv_heads;
        if ((int64_t)pl->layout.units.size() > pl->max_units || pl->layout.n_slots > pl->max_slots)
            return DA_ERR_INVALID_ARG;  // the lengths exceed the declared capacity
        pl->grid = pl->max_units;
    } else {
        pl->max_batch = shape->batch;
        pl->max_slots = pl->layout.n_slots;
        pl->max_units = (int64_t)pl->layout.units.size();
        pl->grid = pl->max_units - pl->layout.n_front_units;   // front units have a launch of their own
    }
    if (pl->grid > 0x7fffffffLL) return DA_ERR_UNSUPPORTED;
    if (pl->max_bins > 0) pl->grid = std::min<int64_t>(pl->grid, pl->max_bins);
    pl->work_grid = pl->grid;
    if (policy->fuse_combine && pl->max_slots > 0) {
        // merge blocks ride behind the attending ones: one per merge task, at most one wave of them
        const int64_t tasks = pl->max_batch * shape->num_kv_heads * combine_slices(shape->head_dim, pl->group);
        pl->grid += std::min<int64_t>(tasks, (int64_t)pl->sm_count * pl->ctas_per_sm);
    }

    pl->workspace_bytes = (size_t)pl->max_slots * shape->num_kv_heads * rec_floats(pl->group, shape->head_dim) * sizeof(float);

    pl->off_units = align_up(sizeof(DevHeader), 32);
    pl->off_seq_info = pl->off_units + align_up((size_t)std::max<int64_t>(pl->max_units, 1) * sizeof(decode_attn_unit_t), 32);
    pl->off_block_begin = pl->off_seq_info + align_up((size_t)std::max<int64_t>(pl->max_batch, 1) * sizeof(SeqInfo), 32);
    pl->off_unit_rank = pl->off_block_begin + align_up((size_t)(pl->grid + 1) * sizeof(int32_t), 32);
    // the binned units by cost rank, for the kernel's redistribution under a RUN mask
    pl->upload_bytes = pl->off_unit_rank +
                       (pl->max_bins > 0
                            ? align_up((size_t)std::max<int64_t>(pl->max_units, 1) * sizeof(int2), 32)
                            : 0);
    pl->off_status = pl->upload_bytes;
    pl->off_tickets = pl->off_status + 32;
    pl->off_queue = pl->off_tickets +
                    align_up(2 * (size_t)std::max<int64_t>(pl->max_batch, 1) * shape->num_kv_heads * sizeof(int32_t), 32);
    pl->total_bytes = pl->off_queue + 32;          // the two counters of the masked launches' queue

    PlanBuffers* pb = new (std::nothrow) PlanBuffers();
    if (!pb) return DA_ERR_INVALID_ARG;
    pl->buffers = pb;
    rc = acquire_buffers(pl->device, pl->total_bytes, pl->total_bytes, pb);
    if (rc != DA_OK) return rc;
    pl->dev = pb->dev;
    pl->pinned = pb->pinned;
    pl->stream = pb->stream;
    pl->upload_done = pb->event;
    pl->launch_done = pb->launched;
    // Buffers that come from a destroyed plan: that plan's last upload has to be out of the pinned
    // mirror before the host rewrites it (long done in practice; a host wait only if not), and its
    // kernels, which may still be running on their caller's stream, have to be done with the device
    // buffer before the new work list lands there (ordered on the device, no host wait).
    DA_CUDA_TRY(cudaEventSynchronize(pl->upload_done));
    DA_CUDA_TRY(cudaStreamWaitEvent(pl->stream, pl->launch_done, 0));
    // one copy: work list, split table, block ranges, and zeros for the status word and tickets
    std::memset(pl->pinned + pl->off_status, 0, pl->total_bytes - pl->off_status);
    fill_host_mirror(pl);
    // The upload is not waited for here: the first launch on a caller's stream is ordered behind it
    // (order_behind_upload), so planning costs no round trip to the device.
    DA_CUDA_TRY(cudaMemcpyAsync(pl->dev, pl->pinned, pl->total_bytes, cudaMemcpyHostToDevice, pl->stream));
    DA_CUDA_TRY(cudaEventRecord(pl->upload_done, pl->stream));
    pl->upload_pending = true;

    if (workspace_bytes_out) *workspace_bytes_out = pl->workspace_bytes;
    *plan_out = pl;
    guard.p = nullptr;
    return DA_OK;
}

int decode_attn_plan_update(decode_attn_plan_t* pl, int32_t batch, const int32_t* seq_lens_host, cudaStream_t stream)
{
    if (!pl || batch < 0 || (batch > 0 && !seq_lens_host)) return DA_ERR_INVALID_ARG;
    if (pl->policy.capacity_batch <= 0) return DA_ERR_UNSUPPORTED;
    if (batch > pl->max_batch) return DA_ERR_INVALID_ARG;
    int64_t total = 0;
    for (int b = 0; b < batch; ++b) total += seq_lens_host[b];
    if (total > pl->policy.capacity_tokens) return DA_ERR_INVALID_ARG;
    decode_attn_shape_t s = pl->shape;
    s.batch = batch;
    Layout lay;
    int rc = make_layout(s, pl->policy, seq_lens_host, pl->sm_count, pl->ctas_per_sm, lay, pl->max_bins);
    if (rc != DA_OK) return rc;
    if ((int64_t)lay.units.size() > pl->max_units || lay.n_slots > pl->max_slots) return DA_ERR_INVALID_ARG;
    // the previous refresh may still be reading the pinned mirror
    DA_CUDA_TRY(cudaEventSynchronize(pl->upload_done));
    pl->upload_pending = false;
    pl->shape.batch = batch;
    pl->layout = std::move(lay);
    pl->seq_lens.assign(seq_lens_host, seq_lens_host + batch);
    fill_host_mirror(pl);
    // the copy is ordered on the caller's stream, behind any launch that still reads the old list
    DA_CUDA_TRY(cudaMemcpyAsync(pl->dev, pl->pinned, pl->upload_bytes, cudaMemcpyHostToDevice, stream));
    DA_CUDA_TRY(cudaEventRecord(pl->upload_done, stream));
    return DA_OK;
}

int decode_attn_plan_get_info(const decode_attn_plan_t* pl, decode_attn_plan_info_t* info)
{
    if (!pl || !info) return DA_ERR_INVALID_ARG;
    std::memset(info, 0, sizeof *info);
    info->n_units = (int64_t)pl->layout.units.size();
    info->grid = pl->grid;
    info->n_slots = pl->layout.n_slots;
    info->workspace_bytes = (int64_t)pl->workspace_bytes;
    info->chunk_tokens = pl->layout.chunk_tokens;
    info->kernel = pl->kernel;
    info->ctas_per_sm = pl->ctas_per_sm;
    info->sm_count = pl->sm_count;
    info->fuse_combine = pl->policy.fuse_combine;
    info->max_splits_used = pl->layout.max_splits_used;
    info->block_threads = pl->block_threads;
    info->dynamic_smem_bytes = pl->dyn_smem;
    return DA_OK;
}

int decode_attn_plan_get_units(const decode_attn_plan_t* pl, decode_attn_unit_t* units_out, int64_t max_units)
{
    if (!pl || !units_out) return DA_ERR_INVALID_ARG;
    if (max_units < (int64_t)pl->layout.units.size()) return DA_ERR_INVALID_ARG;
    std::copy(pl->layout.units.begin(), pl->layout.units.end(), units_out);
    return DA_OK;
}

int decode_attn_plan_check(const decode_attn_plan_t* pl, int32_t batch, const int32_t* seq_lens_host)
{
    if (!pl || (batch > 0 && !seq_lens_host)) return DA_ERR_INVALID_ARG;
    if (batch != pl->shape.batch) return DA_ERR_STALE_PLAN;
    for (int b = 0; b < batch; ++b)
        if (seq_lens_host[b] != pl->seq_lens[b]) return DA_ERR_STALE_PLAN;
    return DA_OK;
}

int decode_attn_plan_destroy(decode_attn_plan_t* pl)
{
    if (!pl) return DA_OK;
    if (pl->buffers) {
        PlanBuffers* pb = static_cast<PlanBuffers*>(pl->buffers);
        release_buffers(*pb);
        delete pb;
    }
    delete pl;
    return DA_OK;
}

// debug_limit > 0: the launch of decode_attn_debug_expire_wait (loads withheld, waits cut short).
static int run_impl(const decode_attn_plan_t* pl, const decode_attn_run_args_t* a, cudaStream_t stream, long long debug_limit)
{
    if (!pl || !a) return DA_ERR_INVALID_ARG;
    // (callers built against the struct without its last two fields pass the shorter size)
    constexpr uint32_t kLegacyArgs = (uint32_t)offsetof(decode_attn_run_args_t, new_k);
    if ((a->struct_size != sizeof(decode_attn_run_args_t) && a->struct_size != kLegacyArgs) || a->flags != 0)
        return DA_ERR_INVALID_ARG;
    decode_attn_run_args_t full;
    std::memset(&full, 0, sizeof full);
    std::memcpy(&full, a, a->struct_size);
    a = &full;
    if ((a->new_k == nullptr) != (a->new_v == nullptr)) return DA_ERR_INVALID_ARG;
    if (a->new_k != nullptr) {
        if (!aligned(a->new_k, 16) || !aligned(a->new_v, 16)) return DA_ERR_INVALID_ARG;
        if (pl->kernel != DA_KERNEL_MMA_TMA || pl->policy.shared_prefix_tokens > 0) return DA_ERR_UNSUPPORTED;
    }
    if (pl->shape.batch == 0 && pl->policy.capacity_batch == 0) return DA_OK;
    if (!a->q || !a->k_cache || !a->v_cache || !a->block_table || !a->seq_lens || !a->out) return DA_ERR_INVALID_ARG;
    if (!aligned(a->q, 16) || !aligned(a->k_cache, 16) || !aligned(a->v_cache, 16) || !aligned(a->out, 16) ||
        !aligned(a->block_table, 4) || !aligned(a->seq_lens, 4))
        return DA_ERR_INVALID_ARG;
    if (pl->workspace_bytes > 0) {
        if (!a->workspace || !aligned(a->workspace, 256)) return DA_ERR_INVALID_ARG;
        if (a->workspace_bytes < pl->workspace_bytes) return DA_ERR_WORKSPACE_TOO_SMALL;
    }
    const bool umma = pl->kernel == DA_KERNEL_UMMA_PREFIX;
    if (pl->grid == 0 && !(umma && pl->layout.n_front_units > 0)) return DA_OK;
    {
        const int rc = order_behind_upload(pl, stream);
        if (rc != DA_OK) return rc;
    }
    KernelParams kp = make_params(pl, *a);
    if (debug_limit > 0) {
        if (pl->kernel != DA_KERNEL_MMA_TMA) return DA_ERR_UNSUPPORTED;
        kp.wait_limit = debug_limit;
        kp.debug_drop_loads = 1;
        kp.hint_first_pages = 0;
    }
    if (pl->kernel == DA_KERNEL_SIMT) {
        simt_kernel_t fn = simt_kernel_for(pl->shape.head_dim, pl->group);
        if (!fn) return DA_ERR_UNSUPPORTED;
        int rc = simt_launch(fn, kp, (unsigned)pl->grid, stream);
        if (rc != DA_OK) return rc;
    } else {
        const unsigned n_front = (unsigned)pl->layout.n_front_units;
        const bool pair = umma && n_front > 0 && pl->grid > 0;
        if (umma && n_front > 0 && !pair) {
            // only shared-prefix units: dealt to one block per SM
            int rc = umma_prefix_launch(pl->shape, pl->group, kp, n_front, std::min<unsigned>(n_front, (unsigned)pl->sm_count),
                                        stream);
            if (rc != DA_OK) return rc;
        }
        if (pl->grid > 0) {
            KernelParams k1 = kp;
            k1.early_trigger = pair;
            int rc = mma_launch(pl->shape, pl->group, k1, (unsigned)pl->grid, stream,
                                pl->policy.shared_prefix_tokens > 0 && !umma);
            if (rc != DA_OK) return rc;
        }
        if (pair) {
            // The bandwidth-bound kernel goes first and the tcgen05 kernel for the shared prefix
            // follows as the second of a pair: its blocks (one per SM, each wanting a whole SM's
            // shared memory) move in as the first kernel's blocks leave, so its start-up and its
            // first tiles fill the other kernel's ragged end instead of following it.
            KernelParams k2 = kp;
            k2.late_wait = 1;
            int rc = umma_prefix_launch(pl->shape, pl->group, k2, n_front, std::min<unsigned>(n_front, (unsigned)pl->sm_count),
                                        stream);
            if (rc != DA_OK) return rc;
        }
    }
    DA_CUDA_TRY(cudaGetLastError());
    mark_launched(pl, stream);
    return DA_OK;
}

int decode_attn_run_ex(const decode_attn_plan_t* pl, const decode_attn_run_args_t* a, cudaStream_t stream)
{
    return run_impl(pl, a, stream, 0);
}

int decode_attn_debug_expire_wait(const decode_attn_plan_t* pl, const decode_attn_run_args_t* a, int64_t limit_cycles,
                                  cudaStream_t stream)
{
    if (limit_cycles <= 0) return DA_ERR_INVALID_ARG;
    // between 50 microseconds and the ordinary limit, whatever was asked for
    const long long limit = std::min<long long>(std::max<long long>(limit_cycles, 100000LL), kWaitLimitCycles);
    return run_impl(pl, a, stream, limit);
}

int decode_attn_run(const decode_attn_plan_t* pl, const void* q, const void* k_cache, const void* v_cache,
                    const int32_t* block_table, const int32_t* seq_lens, void* out, float* lse_or_null,
                    void* workspace, size_t workspace_bytes, cudaStream_t stream)
{
    decode_attn_run_args_t a;
    std::memset(&a, 0, sizeof a);
    a.struct_size = sizeof a;
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache;
    a.block_table = block_table; a.seq_lens = seq_lens;
    a.out = out; a.lse = lse_or_null;
    a.workspace = workspace; a.workspace_bytes = workspace_bytes;
    return decode_attn_run_ex(pl, &a, stream);
}

int decode_attn_combine(const decode_attn_plan_t* pl, const void* workspace, void* out, float* lse_or_null,
                        cudaStream_t stream)
{
    if (!pl || !out) return DA_ERR_INVALID_ARG;
    if (pl->max_slots == 0) return DA_OK;  // nothing was split: run wrote every row
    if (!workspace || !aligned(workspace, 256) || !aligned(out, 16)) return DA_ERR_INVALID_ARG;
    decode_attn_run_args_t a;
    std::memset(&a, 0, sizeof a);
    a.out = out;
    a.lse = lse_or_null;
    a.workspace = const_cast<void*>(workspace);
    const KernelParams kp = make_params(pl, a);
    const unsigned grid = (unsigned)(pl->max_batch * pl->shape.num_kv_heads);
    if (grid == 0) return DA_OK;
    int rc = order_behind_upload(pl, stream);
    if (rc != DA_OK) return rc;
    // a capacity plan may be refreshed to any split count its policy allows
    const int max_splits = pl->policy.capacity_batch > 0 ? kMaxSplits : pl->layout.max_splits_used;
    rc = combine_launch(pl->shape.head_dim, pl->group, kp, grid, stream, max_splits);
    if (rc != DA_OK) return rc;
    DA_CUDA_TRY(cudaGetLastError());
    mark_launched(pl, stream);
    return DA_OK;
}

int decode_attn_merge_shards(const decode_attn_shape_t* shape, int32_t n_shards, const float* out_shards,
                             const float* lse_shards, void* out, float* lse_or_null, cudaStream_t stream)
{
    if (!shape || !out_shards || !lse_shards || !out) return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    if (n_shards < 1 || n_shards > kMaxSplits) return DA_ERR_INVALID_ARG;
    if (!aligned(out_shards, 16) || !aligned(out, 16) || !aligned(lse_shards, 4)) return DA_ERR_INVALID_ARG;
    const int64_t rows = (int64_t)shape->batch * shape->num_q_heads;
    if (rows == 0) return DA_OK;
    const int D4 = shape->head_dim / 4;
    const int64_t threads = rows * D4;
    const int64_t blocks = (threads + 127) / 128;
    if (blocks > 0x7fffffffLL) return DA_ERR_UNSUPPORTED;
    decode_attn_merge_shards_kernel<<<(unsigned)blocks, 128, 0, stream>>>(out_shards, lse_shards, n_shards, rows, D4, out,
                                                                            lse_or_null, out_kind_of(shape->out_dtype));
    DA_CUDA_TRY(cudaGetLastError());
    return DA_OK;
}

static int static_step_status(cudaStream_t stream);

int decode_attn_last_device_status(const decode_attn_plan_t* pl, cudaStream_t stream)
{
    if (!pl) return static_step_status(stream);     // the allocation-free step has no plan: its status word
    int32_t st = 0;
    DA_CUDA_TRY(cudaEventSynchronize(pl->upload_done));
    pl->upload_pending = false;
    DA_CUDA_TRY(cudaStreamSynchronize(stream));
    DA_CUDA_TRY(cudaMemcpy(&st, pl->dev + pl->off_status, sizeof st, cudaMemcpyDeviceToHost));
    if (st != 0) {
        DA_CUDA_TRY(cudaMemset(pl->dev + pl->off_status, 0, sizeof(int32_t)));
        // a failed launch may have left tickets half drawn
        DA_CUDA_TRY(cudaMemset(pl->dev + pl->off_tickets, 0, pl->total_bytes - pl->off_tickets));
    }
    return st;
}

int decode_attn_validate_block_table(const decode_attn_shape_t* shape, const int32_t* seq_lens_host,
                                     const int32_t* block_table_host)
{
    if (!shape || (shape->batch > 0 && (!seq_lens_host || !block_table_host))) return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    for (int b = 0; b < shape->batch; ++b) {
        if (seq_lens_host[b] < 0) return DA_ERR_INVALID_ARG;
        const int64_t pages = ((int64_t)seq_lens_host[b] + shape->page_size - 1) / shape->page_size;
        if (pages > shape->max_pages_per_seq) return DA_ERR_INVALID_ARG;
        for (int64_t i = 0; i < pages; ++i) {
            const int32_t pg = block_table_host[(int64_t)b * shape->max_pages_per_seq + i];
            if (pg < 0 || pg >= shape->num_pages) return DA_ERR_BAD_PAGE;
        }
    }
    return DA_OK;
}

int decode_attn_validate_shared_prefix(const decode_attn_shape_t* shape, int32_t shared_prefix_tokens,
                                       const int32_t* seq_lens_host, const int32_t* block_table_host)
{
    if (!shape || shared_prefix_tokens < 0 || (shape->batch > 0 && (!seq_lens_host || !block_table_host)))
        return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    if (shared_prefix_tokens % shape->page_size != 0) return DA_ERR_INVALID_ARG;
    const int64_t pages = shared_prefix_tokens / shape->page_size;
    if (pages > shape->max_pages_per_seq) return DA_ERR_INVALID_ARG;
    for (int b = 0; b < shape->batch; ++b) {
        if (seq_lens_host[b] < shared_prefix_tokens) return DA_ERR_INVALID_ARG;
        for (int64_t i = 0; i < pages; ++i)
            if (block_table_host[(int64_t)b * shape->max_pages_per_seq + i] != block_table_host[i]) return DA_ERR_BAD_PAGE;
    }
    return DA_OK;
}

int decode_attn_debug_gather(const decode_attn_plan_t* pl, int32_t seq, const void* k_cache, const void* v_cache,
                             const int32_t* block_table, void* k_out, void* v_out, cudaStream_t stream)
{
    if (!pl || !k_cache || !v_cache || !block_table || !k_out || !v_out) return DA_ERR_INVALID_ARG;
    if (seq < 0 || seq >= pl->shape.batch) return DA_ERR_INVALID_ARG;
    if (pl->policy.shared_prefix_tokens > 0) return DA_ERR_UNSUPPORTED;
    if (!aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(k_out, 16) || !aligned(v_out, 16))
        return DA_ERR_INVALID_ARG;
    if (pl->grid == 0) return DA_OK;
    decode_attn_run_args_t a;
    std::memset(&a, 0, sizeof a);
    a.k_cache = k_cache; a.v_cache = v_cache; a.block_table = block_table;
    const KernelParams kp = make_params(pl, a);
    if (pl->kernel == DA_KERNEL_UMMA_PREFIX) return DA_ERR_UNSUPPORTED;
    if (order_behind_upload(pl, stream) != DA_OK) return DA_ERR_CUDA;
    mma_launch_guard guard{pl, stream};
    return mma_debug_gather(pl->shape, pl->group, kp, seq, k_out, v_out, (unsigned)pl->work_grid, stream);
}

int decode_attn_gather_probe(const decode_attn_plan_t* pl, const void* k_cache, const void* v_cache,
                             const int32_t* block_table, uint32_t* checksum_out, cudaStream_t stream)
{
    if (!pl || !k_cache || !v_cache || !block_table || !checksum_out) return DA_ERR_INVALID_ARG;
    if (!aligned(k_cache, 16) || !aligned(v_cache, 16)) return DA_ERR_INVALID_ARG;
    if (pl->policy.shared_prefix_tokens > 0) return DA_ERR_UNSUPPORTED;
    if (pl->grid == 0) return DA_OK;
    decode_attn_run_args_t a;
    std::memset(&a, 0, sizeof a);
    a.k_cache = k_cache; a.v_cache = v_cache; a.block_table = block_table;
    const KernelParams kp = make_params(pl, a);
    if (order_behind_upload(pl, stream) != DA_OK) return DA_ERR_CUDA;
    mma_launch_guard guard{pl, stream};
    return mma_gather_probe(pl->shape, pl->group, kp, checksum_out, (unsigned)pl->layout.units.size(), (unsigned)pl->work_grid,
                            stream);
}

static int append_impl(const decode_attn_shape_t* shape, int32_t* status, const void* new_k, const void* new_v,
                       const int32_t* block_table, const int32_t* seq_lens, void* k_cache, void* v_cache,
                       cudaStream_t stream)
{
    if (!shape || !new_k || !new_v || !block_table || !seq_lens || !k_cache || !v_cache) return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    if (!aligned(new_k, 16) || !aligned(new_v, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16))
        return DA_ERR_INVALID_ARG;
    if (shape->batch == 0) return DA_OK;
    AppendParams ap;
    std::memset(&ap, 0, sizeof ap);
    ap.new_k = static_cast<const __nv_bfloat16*>(new_k);
    ap.new_v = static_cast<const __nv_bfloat16*>(new_v);
    ap.k = static_cast<__nv_bfloat16*>(k_cache);
    ap.v = static_cast<__nv_bfloat16*>(v_cache);
    ap.block_table = block_table;
    ap.seq_lens = seq_lens;
    ap.status = status;
    ap.k_stride_page = shape->k_stride_page; ap.k_stride_token = shape->k_stride_token; ap.k_stride_head = shape->k_stride_head;
    ap.v_stride_page = shape->v_stride_page; ap.v_stride_token = shape->v_stride_token; ap.v_stride_head = shape->v_stride_head;
    ap.num_pages = shape->num_pages;
    ap.batch = shape->batch;
    ap.num_kv_heads = shape->num_kv_heads;
    ap.head_dim = shape->head_dim;
    ap.max_pages_per_seq = shape->max_pages_per_seq;
    ap.page_shift = log2_of(shape->page_size);
    const int rows = shape->batch * shape->num_kv_heads;
    const unsigned grid = (unsigned)((rows + kAppendThreads / 32 - 1) / (kAppendThreads / 32));
    cudaLaunchConfig_t cfg;
    cfg.gridDim = dim3(grid, 1, 1);
    cfg.blockDim = dim3(kAppendThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, decode_attn_append_kernel, ap) != cudaSuccess) {
        (void)cudaGetLastError();
        return DA_ERR_CUDA;
    }
    return DA_OK;
}

int decode_attn_append_kv(const decode_attn_shape_t* shape, const void* new_k, const void* new_v,
                          const int32_t* block_table, const int32_t* seq_lens, void* k_cache, void* v_cache,
                          cudaStream_t stream)
{
    return append_impl(shape, nullptr, new_k, new_v, block_table, seq_lens, k_cache, v_cache, stream);
}

int decode_attn_append_kv_checked(const decode_attn_plan_t* pl, const void* new_k, const void* new_v,
                                  const int32_t* block_table, const int32_t* seq_lens, void* k_cache, void* v_cache,
                                  cudaStream_t stream)
{
    if (!pl) return DA_ERR_INVALID_ARG;
    int rc = order_behind_upload(pl, stream);      // the upload also zeroes the status word this launch may write
    if (rc != DA_OK) return rc;
    rc = append_impl(&pl->shape, reinterpret_cast<int32_t*>(pl->dev + pl->off_status), new_k, new_v, block_table,
                     seq_lens, k_cache, v_cache, stream);
    if (rc == DA_OK) mark_launched(pl, stream);
    return rc;
}

// ------------------------------------------------------------------ host-buffer step

namespace {
struct HostArena {
    std::mutex mu;
    int device = -1;
    char* base = nullptr;
    size_t bytes = 0;
} g_arena;
}  // namespace

int decode_attn_host_release(void)
{
    std::lock_guard<std::mutex> lock(g_arena.mu);
    if (g_arena.base) {
        cudaFree(g_arena.base);
        (void)cudaGetLastError();
    }
    g_arena.base = nullptr;
    g_arena.bytes = 0;
    g_arena.device = -1;
    std::lock_guard<std::mutex> lock2(g_buffers.mu);
    for (PlanBuffers& b : g_buffers.free_list) free_buffers(b);
    g_buffers.free_list.clear();
    return DA_OK;
}

int decode_attn_host_step(const decode_attn_shape_t* shape, const decode_attn_policy_t* policy, const void* q_host,
                          const void* k_cache_host, const void* v_cache_host, int64_t pool_elems,
                          const int32_t* block_table_host, const int32_t* seq_lens_host, void* out_host,
                          float* lse_host_or_null)
{
    if (!shape || !policy || !q_host || !k_cache_host || !v_cache_host || !block_table_host || !seq_lens_host ||
        !out_host || pool_elems <= 0)
        return DA_ERR_INVALID_ARG;
    if (policy->capacity_batch != 0) return DA_ERR_INVALID_ARG;
    int rc = decode_attn_validate_block_table(shape, seq_lens_host, block_table_host);
    if (rc != DA_OK) return rc;
    if (shape->batch == 0) return DA_OK;

    decode_attn_plan_t* plan = nullptr;
    size_t ws_bytes = 0;
    rc = decode_attn_plan(shape, policy, seq_lens_host, &plan, &ws_bytes);
    if (rc != DA_OK) return rc;
    struct PlanGuard {
        decode_attn_plan_t* p;
        ~PlanGuard() { decode_attn_plan_destroy(p); }
    } pg{plan};

    const size_t out_elem = shape->out_dtype == DA_DTYPE_FP32 ? 4 : 2;
    const size_t q_bytes = (size_t)shape->batch * shape->num_q_heads * shape->head_dim * 2;
    const size_t pool_bytes = (size_t)pool_elems * 2;
    const size_t bt_bytes = (size_t)shape->batch * shape->max_pages_per_seq * 4;
    const size_t sl_bytes = (size_t)shape->batch * 4;
    const size_t out_bytes = (size_t)shape->batch * shape->num_q_heads * shape->head_dim * out_elem;
    const size_t lse_bytes = (size_t)shape->batch * shape->num_q_heads * 4;
    size_t off = 0;
    auto take = [&off](size_t n) { size_t o = off; off = align_up(off + n, 256); return o; };
    const size_t o_q = take(q_bytes), o_k = take(pool_bytes), o_v = take(pool_bytes), o_bt = take(bt_bytes),
                 o_sl = take(sl_bytes), o_out = take(out_bytes), o_lse = take(lse_bytes), o_ws = take(ws_bytes);

    std::lock_guard<std::mutex> lock(g_arena.mu);
    int dev = -1;
    DA_CUDA_TRY(cudaGetDevice(&dev));
    if (g_arena.device != dev || g_arena.bytes < off) {
        if (g_arena.base) cudaFree(g_arena.base);
        g_arena.base = nullptr;
        g_arena.bytes = 0;
        DA_CUDA_TRY(cudaMalloc(&g_arena.base, off));
        g_arena.bytes = off;
        g_arena.device = dev;
    }
    char* A = g_arena.base;
    cudaStream_t st = plan->stream;
    DA_CUDA_TRY(cudaMemcpyAsync(A + o_q, q_host, q_bytes, cudaMemcpyHostToDevice, st));
    DA_CUDA_TRY(cudaMemcpyAsync(A + o_k, k_cache_host, pool_bytes, cudaMemcpyHostToDevice, st));
    DA_CUDA_TRY(cudaMemcpyAsync(A + o_v, v_cache_host, pool_bytes, cudaMemcpyHostToDevice, st));
    DA_CUDA_TRY(cudaMemcpyAsync(A + o_bt, block_table_host, bt_bytes, cudaMemcpyHostToDevice, st));
    DA_CUDA_TRY(cudaMemcpyAsync(A + o_sl, seq_lens_host, sl_bytes, cudaMemcpyHostToDevice, st));
    float* lse_dev = lse_host_or_null ? reinterpret_cast<float*>(A + o_lse) : nullptr;
    rc = decode_attn_run(plan, A + o_q, A + o_k, A + o_v, reinterpret_cast<const int32_t*>(A + o_bt),
                         reinterpret_cast<const int32_t*>(A + o_sl), A + o_out, lse_dev, ws_bytes ? A + o_ws : nullptr,
                         ws_bytes, st);
    if (rc != DA_OK) return rc;
    if (!policy->fuse_combine) {
        rc = decode_attn_combine(plan, ws_bytes ? A + o_ws : nullptr, A + o_out, lse_dev, st);
        if (rc != DA_OK) return rc;
    }
    DA_CUDA_TRY(cudaMemcpyAsync(out_host, A + o_out, out_bytes, cudaMemcpyDeviceToHost, st));
    if (lse_host_or_null)
        DA_CUDA_TRY(cudaMemcpyAsync(lse_host_or_null, A + o_lse, lse_bytes, cudaMemcpyDeviceToHost, st));
    return decode_attn_last_device_status(plan, st);
}

const char* decode_attn_strerror(int status)
{
    switch (status) {
        case DA_OK: return "ok";
        case DA_ERR_INVALID_ARG: return "invalid argument";
        case DA_ERR_UNSUPPORTED: return "unsupported shape, dtype or policy";
        case DA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case DA_ERR_STALE_PLAN: return "plan is stale: seq_lens differ from the planned lengths";
        case DA_ERR_CUDA: return "CUDA call failed or no CUDA device";
        case DA_ERR_BAD_PAGE: return "block table refers to a page outside the pool";
        case DA_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        default: return "unknown status";
    }
}

const char* decode_attn_version(void) { return "0.1 sm_100a"; }

// ------------------------------------------------------------------ allocation-free step
//
// Scratch for decode_attn_step_static: work list, per-sequence split table,
// status word and partial records, all inside one file-scope device array.
// Every GPU that loads this library holds these bytes until the process ends.
constexpr size_t kStaticScratchBytes = 8u << 20;       // 8 MiB
constexpr int kStaticMaxUnits = 4096;
constexpr int kStaticMaxBatch = 1024;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

// header | split table | work list | status word | records.  The split table sits in front of the
// work list so that each of the two uploads is as long as the step needs and no longer.
constexpr size_t kStaticOffSeqInfo = 256;
constexpr size_t kStaticOffUnits = kStaticOffSeqInfo + sizeof(SeqInfo) * kStaticMaxBatch;
constexpr size_t kStaticOffStatus = kStaticOffUnits + sizeof(decode_attn_unit_t) * kStaticMaxUnits;
constexpr size_t kStaticOffRecords = kStaticOffStatus + 256;
static_assert(kStaticOffRecords % 256 == 0 && kStaticOffRecords < kStaticScratchBytes, "static scratch layout");

struct StaticSetup {
    std::mutex mu;
    static constexpr int kMaxDevices = 64;
    unsigned char* base[kMaxDevices] = {};      // device address of g_static_scratch, per device
    int sm_count[kMaxDevices] = {};
    // host copy of the upload region; calls are serialised by `mu` while it is filled and enqueued
    alignas(16) unsigned char staging[kStaticOffStatus];
} g_static;

}  // namespace

// Status word of decode_attn_step_static on the current device: synchronises `stream`, returns the
// worst condition its kernels recorded since the last call and clears it.  Copies through the
// static array's address; allocates nothing.
static int static_step_status(cudaStream_t stream)
{
    int dev = -1;
    DA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= StaticSetup::kMaxDevices) return DA_ERR_UNSUPPORTED;
    unsigned char* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static.mu);
        base = g_static.base[dev];
    }
    if (base == nullptr) return DA_OK;              // no static step has run on this device yet
    int32_t st = 0;
    DA_CUDA_TRY(cudaStreamSynchronize(stream));
    DA_CUDA_TRY(cudaMemcpy(&st, base + kStaticOffStatus, sizeof st, cudaMemcpyDeviceToHost));
    if (st != 0) DA_CUDA_TRY(cudaMemset(base + kStaticOffStatus, 0, sizeof(int32_t)));
    return st;
}

int decode_attn_step_static(const decode_attn_shape_t* shape, const int32_t* seq_lens_host, const void* q,
                            const void* k_cache, const void* v_cache, const int32_t* block_table,
                            const int32_t* seq_lens, void* out, float* lse_or_null, cudaStream_t stream)
{
    if (!shape || !q || !k_cache || !v_cache || !block_table || !seq_lens || !out) return DA_ERR_INVALID_ARG;
    if (shape->batch > 0 && !seq_lens_host) return DA_ERR_INVALID_ARG;
    int rc = validate_shape(*shape);
    if (rc != DA_OK) return rc;
    if (!aligned(q, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) || !aligned(out, 16)) return DA_ERR_INVALID_ARG;
    if (shape->batch == 0) return DA_OK;
    if (shape->batch > kStaticMaxBatch) return DA_ERR_WORKSPACE_TOO_SMALL;
    // Every call plans on the host and uploads its own work list, so a captured call would replay
    // a stale one: refuse instead.
    if (stream_is_capturing(stream)) return DA_ERR_UNSUPPORTED;

    decode_attn_policy_t policy;
    std::memset(&policy, 0, sizeof policy);
    policy.split_mode = DA_SPLIT_DETERMINISTIC;     // boundaries from the lengths alone: no device query needed
    const int G = shape->num_q_heads / shape->num_kv_heads;
    const int kernel = pick_kernel(*shape, policy);

    int dev = -1;
    DA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= StaticSetup::kMaxDevices) return DA_ERR_UNSUPPORTED;

    std::lock_guard<std::mutex> lock(g_static.mu);
    if (g_static.base[dev] == nullptr) {
        // First call on this device (make it before any stream capture): in host code the
        // array's name is only a stand-in, so ask the runtime for its address on the current
        // device.  Also done once here: the kernels' shared-memory opt-in.
        void* ptr = nullptr;
        DA_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_scratch));
        int block_threads = 0, dyn_smem = 0;
        if (query_occupancy(kernel, shape->head_dim, G, &block_threads, &dyn_smem) <= 0) return DA_ERR_CUDA;
        DA_CUDA_TRY(cudaDeviceGetAttribute(&g_static.sm_count[dev], cudaDevAttrMultiProcessorCount, dev));
        // (a __device__ array without an initialiser starts zeroed: the status word reads DA_OK)
        g_static.base[dev] = static_cast<unsigned char*>(ptr);
    } else if (kernel == DA_KERNEL_MMA_TMA) {
        int block_threads = 0, dyn_smem = 0;       // another head_dim / group may need its own opt-in
        if (query_occupancy(kernel, shape->head_dim, G, &block_threads, &dyn_smem) <= 0) return DA_ERR_CUDA;
    }
    unsigned char* const base = g_static.base[dev];

    Layout lay;
    rc = make_layout(*shape, policy, seq_lens_host, g_static.sm_count[dev], 1, lay);
    if (rc != DA_OK) return rc;
    const size_t rec_bytes = (size_t)rec_floats(G, shape->head_dim) * sizeof(float);
    if (lay.units.size() > (size_t)kStaticMaxUnits ||
        (size_t)lay.n_slots * shape->num_kv_heads * rec_bytes > kStaticScratchBytes - kStaticOffRecords)
        return DA_ERR_WORKSPACE_TOO_SMALL;          // the step does not fit the built-in scratch

    // upload region: header, units, split table (host copy lives in g_static.staging)
    DevHeader* hdr = reinterpret_cast<DevHeader*>(g_static.staging);
    hdr->n_units = (int32_t)lay.units.size();
    hdr->batch = shape->batch;
    hdr->n_ranked = 0;
    hdr->first_binned = 0;
    std::memcpy(g_static.staging + kStaticOffUnits, lay.units.data(), lay.units.size() * sizeof(decode_attn_unit_t));
    SeqInfo* si = reinterpret_cast<SeqInfo*>(g_static.staging + kStaticOffSeqInfo);
    for (int b = 0; b < shape->batch; ++b) {
        si[b].slot_base = lay.slot_base[b];
        si[b].n_splits = lay.splits[b];
        si[b].seq_len = seq_lens_host[b];
        si[b].pad = 0;
    }
    // The array keeps the previous call's contents.  What the kernels only read is overwritten by
    // the two uploads below, records are written before they are read, and the status word is
    // cumulative on purpose (decode_attn_last_device_status(NULL, ...) reads and clears it), so
    // nothing needs zeroing here.
    // Pageable source: the runtime has taken the bytes when the call returns, so the staging area
    // may be reused by the next call.
    DA_CUDA_TRY(cudaMemcpyAsync(base, g_static.staging, kStaticOffSeqInfo + sizeof(SeqInfo) * (size_t)shape->batch,
                                cudaMemcpyHostToDevice, stream));
    DA_CUDA_TRY(cudaMemcpyAsync(base + kStaticOffUnits, g_static.staging + kStaticOffUnits,
                                lay.units.size() * sizeof(decode_attn_unit_t), cudaMemcpyHostToDevice, stream));

    KernelParams kp;
    std::memset(&kp, 0, sizeof kp);
    kp.q = static_cast<const __nv_bfloat16*>(q);
    kp.k = static_cast<const __nv_bfloat16*>(k_cache);
    kp.v = static_cast<const __nv_bfloat16*>(v_cache);
    kp.block_table = block_table;
    kp.seq_lens = seq_lens;
    kp.out = out;
    kp.lse = lse_or_null;
    kp.ws = reinterpret_cast<float*>(base + kStaticOffRecords);
    kp.header = reinterpret_cast<const DevHeader*>(base);
    kp.units = reinterpret_cast<const decode_attn_unit_t*>(base + kStaticOffUnits);
    kp.seq_info = reinterpret_cast<const SeqInfo*>(base + kStaticOffSeqInfo);
    kp.tickets = nullptr;                           // only fused plans count arrivals; this step is not one
    kp.status = reinterpret_cast<int32_t*>(base + kStaticOffStatus);
    kp.k_stride_page = shape->k_stride_page; kp.k_stride_token = shape->k_stride_token; kp.k_stride_head = shape->k_stride_head;
    kp.v_stride_page = shape->v_stride_page; kp.v_stride_token = shape->v_stride_token; kp.v_stride_head = shape->v_stride_head;
    kp.num_pages = shape->num_pages;
    kp.num_q_heads = shape->num_q_heads;
    kp.num_kv_heads = shape->num_kv_heads;
    kp.max_pages_per_seq = shape->max_pages_per_seq;
    const float scale = shape->sm_scale > 0.f ? shape->sm_scale : 1.0f / sqrtf((float)shape->head_dim);
    kp.scale_log2 = scale * kLog2e;
    kp.out_kind = out_kind_of(shape->out_dtype);
    kp.in_f16 = shape->kv_dtype == DA_DTYPE_FP16;
    kp.tile_shift = log2_of(shape->page_size) - 4;
    kp.fused = 0;
    kp.grid_exit = 0;
    kp.wait_limit = kWaitLimitCycles;
    kp.n_units = (int32_t)lay.units.size();
    kp.n_work_blocks = (int32_t)lay.units.size();
    kp.batch = shape->batch;

    const unsigned grid = (unsigned)lay.units.size();
    if (kernel == DA_KERNEL_SIMT) {
        simt_kernel_t fn = simt_kernel_for(shape->head_dim, G);
        if (!fn) return DA_ERR_UNSUPPORTED;
        rc = simt_launch(fn, kp, grid, stream);
        if (rc != DA_OK) return rc;
    } else {
        rc = mma_launch(*shape, G, kp, grid, stream);
        if (rc != DA_OK) return rc;
    }
    DA_CUDA_TRY(cudaGetLastError());
    if (lay.n_slots > 0) {
        rc = combine_launch(shape->head_dim, G, kp, (unsigned)(shape->batch * shape->num_kv_heads), stream,
                            lay.max_splits_used);
        if (rc != DA_OK) return rc;
        DA_CUDA_TRY(cudaGetLastError());
    }
    return DA_OK;
}

#ifdef DA_TRACE
// Debug builds only: device buffer of 32 uint64 stamps per block (NULL switches tracing off).
int decode_attn_trace_set_buffer(unsigned long long* device_buffer)
{
    g_trace_buffer = device_buffer;
    return DA_OK;
}
#endif

}  // extern "C"
