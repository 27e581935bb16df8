// kaitian.cu -- the device side of the C ABI for KAITIAN's hierarchical, load-weighted gradient
// synchronisation (paper Sections III-A and III-C): contexts and weights, device tables,
// launches, pinned-host staging, the broadcast, recorded steps, memory shared between processes,
// the entry point that allocates nothing.  The kernels are in kt_kernels.cuh, the entry points
// that are pure host arithmetic (scheduler, plan, share ranges, host barrier ...) in kt_host.cu;
// the contract of every entry point is in include/kaitian.h.
//
// Data layout in device memory
//   gradients   K*T caller-owned tensors (fp32 or bf16), read in place through a pointer
//               table [K][T] kept in group-major rank order and transport tensor order
//   transport   G caller-owned fp32 buffers of transport_numel elements: tensors laid end
//               to end in reverse list order, each at a multiple of 8 elements, buckets at
//               multiples of 64, zero padding in the gaps
//   tensor table  one 32-byte record per tensor (transport offset, numel, numel + padding,
//               flags) and a prefix sum of TILE-sized work units per tensor
//
// One rank per device (kt_shard_bind): the same tables, but the pointer table holds the M
// members of the rank's group only (its own tensors and its mates' peer-mapped ones), and every
// launch and copy covers the member's share of the range: a contiguous run of work units
// (unit_range), which is one contiguous element range of the transport (unit_start).

#include "../../include/kaitian.h"

#include <cuda.h>            // types and enumerators only: driver entry points are asked of the runtime
#include <cuda_runtime.h>

#include "kt_kernels.cuh"
#include "kt_internal.h"

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdarg>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <thread>
#include <utility>
#include <vector>

using namespace ktd;

namespace {

// Makes a context's device current for the length of a call and puts the caller's device back
// afterwards: a library call must not change which device the calling thread works on.
struct DeviceScope {
    int prev = -1;
    cudaError_t status = cudaSuccess;
    explicit DeviceScope(int device) {
        status = cudaGetDevice(&prev);
        if (status == cudaSuccess && prev != device) status = cudaSetDevice(device);
        else if (status == cudaSuccess) prev = -1;          // nothing to restore
    }
    ~DeviceScope() {
        if (prev >= 0) cudaSetDevice(prev);
    }
    DeviceScope(const DeviceScope &) = delete;
    DeviceScope &operator=(const DeviceScope &) = delete;
};

#define KT_ON_DEVICE(dev)                                                                   \
    DeviceScope device_scope_(dev);                                                         \
    if (device_scope_.status != cudaSuccess)                                                \
        return fail(KT_ERR_CUDA, "selecting device %d: %s", (dev), cudaGetErrorString(device_scope_.status))

// ------------------------------------------------------------------ host-side state
struct StageSlot {
    cudaEvent_t done = nullptr;
    bool recorded = false;
};

// One destination table of kt_unpack_scale / kt_sync_direct: R*T output pointers in transport
// tensor order, then one flag per tensor (all R destinations 16-byte aligned).  A context keeps
// several, so that a caller that alternates between sets of output tensors (double-buffered
// gradients) finds each set already on the device.
constexpr int KT_OUT_SETS = 8;
struct OutSet {
    void *dev = nullptr;             // device table
    char *staging = nullptr;         // pinned host image the upload reads
    size_t cap = 0;                  // bytes of both
    std::vector<void *> ptrs;        // what was uploaded (caller's order)
    int R = 0, dtype = -1;
    cudaEvent_t uploaded = nullptr;  // the upload has read the staging image and written the table
    cudaStream_t upload_stream = nullptr;   // where that copy was queued
    cudaEvent_t used = nullptr;      // the last kernel that reads the device table
    uint64_t stamp = 0;              // last use, for replacement
    bool in_recording = false;       // a recorded step reads this table whenever it is replayed: never replaced
};

}  // namespace

struct kt_ctx {
    int device = 0;
    int sm_count = 0;
    int K = 0, G = 0;
    std::vector<int32_t> group_of, shares;
    std::vector<int> order;          // group-major rank order
    RankTab rt{};
    GroupTab gt{};

    // plan (valid once planned)
    bool planned = false;
    int T = 0;
    int in_dtype = KT_F32;
    int transport_dtype = KT_F32;                    // element type of the transport buffers
    int tile = TILE_F32;                             // elements per work unit (by gradient dtype)
    std::vector<int64_t> numel, tensor_offset;       // user tensor order
    std::vector<int32_t> bucket_of;
    std::vector<int64_t> bucket_start, bucket_numel;
    std::vector<int> bucket_u_lo, bucket_u_hi;       // transport-order tensor range per bucket
    int64_t transport_numel = 0;
    std::vector<int> prefix;                         // [T+1], transport order
    std::vector<TInfo> info;                         // [T], transport order

    // device tables
    void *d_tables = nullptr;        // one allocation: prefix | info | grad ptrs
    size_t d_tables_bytes = 0;
    int *d_prefix = nullptr;
    TInfo *d_info = nullptr;
    const void **d_ptrs = nullptr;
    std::vector<const void *> h_ptrs;   // the registered gradient pointers, [K][T] as the caller listed them
    OutSet out_sets[KT_OUT_SETS];    // destination tables on the device, least recently used replaced
    uint64_t out_clock = 0;
    bool recording_broken = false;   // a call between kt_graph_begin and kt_graph_end could not be recorded

    // one rank per device (kt_shard_bind): this context belongs to rank `shard_rank`, member
    // `shard_member` of the `shard_M` ranks of group `shard_g`; it works on that member's share
    // of every range and reads the gradients of its group's members only
    int shard_rank = -1, shard_g = 0, shard_member = 0, shard_M = 0;
    RankTab shard_rt{};              // the group's members alone, in ascending rank order

    cudaEvent_t ev_main = nullptr;
    std::vector<StageSlot> slots[2]; // per direction: index 0 = all buckets, 1 + b = bucket b
    std::vector<cudaEvent_t> chunk_events;   // chunk k went down: its way up may start
    int64_t launches = 0;
    std::vector<std::pair<const void *, int>> occupancy;   // resident CTAs per SM, per kernel
};

namespace {

bool sharded(const kt_ctx *c) { return c->shard_rank >= 0; }
// how many ranks' gradient tensors a context reads: all of them, or its own group's
int n_sources(const kt_ctx *c) { return sharded(c) ? c->shard_M : c->K; }
// which of the caller's rank lists feeds position k of the device pointer table
int source_of(const kt_ctx *c, int k) { return sharded(c) ? k : c->order[k]; }
const RankTab &reduce_table(const kt_ctx *c) { return sharded(c) ? c->shard_rt : c->rt; }

// The group's own rows of the rank table, for a context bound to one rank.
void refresh_shard(kt_ctx *c) {
    if (!sharded(c)) return;
    std::memset(&c->shard_rt, 0, sizeof(c->shard_rt));
    int m = 0;
    for (int k = 0; k < c->K; ++k) {
        if (c->rt.gid[k] != c->shard_g) continue;
        c->shard_rt.coef[m] = c->rt.coef[k];
        c->shard_rt.gid[m] = static_cast<signed char>(c->shard_g);
        ++m;
    }
    c->shard_rt.first[0] = 1;
    c->shard_rt.last[m - 1] = 1;
    c->shard_rt.K = m;
}

int compute_coefficients(kt_ctx *c) {
    std::vector<int64_t> Bg(c->G, 0);
    int64_t B = 0;
    for (int r = 0; r < c->K; ++r) {
        Bg[c->group_of[r]] += c->shares[r];
        B += c->shares[r];
    }
    c->order.clear();
    for (int g = 0; g < c->G; ++g)
        for (int r = 0; r < c->K; ++r)
            if (c->group_of[r] == g) c->order.push_back(r);
    std::memset(&c->rt, 0, sizeof(c->rt));
    c->rt.K = c->K;
    for (int k = 0; k < c->K; ++k) {
        const int r = c->order[k];
        const int g = c->group_of[r];
        c->rt.coef[k] = static_cast<float>(static_cast<double>(c->shares[r]) / static_cast<double>(Bg[g]));
        c->rt.gid[k] = static_cast<signed char>(g);
        c->rt.first[k] = (k == 0 || c->group_of[c->order[k - 1]] != g);
        c->rt.last[k] = (k == c->K - 1 || c->group_of[c->order[k + 1]] != g);
    }
    std::memset(&c->gt, 0, sizeof(c->gt));
    c->gt.G = c->G;
    for (int g = 0; g < c->G; ++g)
        c->gt.W[g] = static_cast<float>(static_cast<double>(Bg[g]) / static_cast<double>(B));
    refresh_shard(c);
    return KT_OK;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename P>
int all_aligned32(P *const *bufs, int n) {
    for (int i = 0; i < n; ++i)
        if (reinterpret_cast<uintptr_t>(bufs[i]) & 31u) return 0;
    return 1;
}

// Grid of a grid-stride kernel: one wave of resident CTAs (SM count x occupancy), or
// fewer when there is less work.  Occupancy is queried once per kernel and cached.
template <typename Kern>
int grid_for(kt_ctx *c, Kern kernel, size_t smem, long long units) {
    const void *key = reinterpret_cast<const void *>(kernel);
    int per_sm = 0;
    for (const auto &kv : c->occupancy)
        if (kv.first == key) per_sm = kv.second;
    if (!per_sm) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, NT, smem) != cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            per_sm = 1;
        }
        c->occupancy.emplace_back(key, per_sm);
    }
    const long long cap = static_cast<long long>(c->sm_count) * per_sm;
    const long long g = units < cap ? units : cap;
    return static_cast<int>(g < 1 ? 1 : g);
}

// Work units [*t0, *t1) of a call's range (one bucket, or everything for bucket == -1) that the
// context works on: all of them, or, bound to one rank, that member's share.
void unit_range(const kt_ctx *c, int bucket, int member, int *t0, int *t1) {
    const int u_lo = bucket < 0 ? 0 : c->bucket_u_lo[bucket];
    const int u_hi = bucket < 0 ? c->T : c->bucket_u_hi[bucket];
    *t0 = c->prefix[u_lo];
    *t1 = c->prefix[u_hi];
    if (member >= 0) {
        int64_t first, past;
        member_units(*t1 - *t0, member, c->shard_M, &first, &past);
        *t1 = *t0 + static_cast<int>(past);
        *t0 = *t0 + static_cast<int>(first);
    }
}

// The tensor (transport order) that holds work unit `tile`; T for the index past the last unit.
int tensor_of_unit(const kt_ctx *c, int tile) {
    return static_cast<int>(std::upper_bound(c->prefix.begin(), c->prefix.end(), tile) - c->prefix.begin()) - 1;
}

// First transport element of a work unit; transport_numel for the index past the last unit.
// Tensors follow one another without gaps (a tensor's extent includes the padding behind it),
// so a run of units is one contiguous element range.
int64_t unit_start(const kt_ctx *c, int tile) {
    const int u = tensor_of_unit(c, tile);
    if (u >= c->T) return c->transport_numel;
    return c->info[u].dst_off + static_cast<int64_t>(tile - c->prefix[u]) * c->tile;
}

// tile range of a bucket (or of everything for bucket == -1)
// whole: the full range even on a context bound to one rank (the root of a broadcast sends
// everything, not a share)
int make_tile_plan(const kt_ctx *c, int bucket, TilePlan *tp, bool whole = false) {
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range [-1, %d)", bucket, (int)c->bucket_start.size());
    const bool share = sharded(c) && !whole;
    int t0, t1;
    unit_range(c, bucket, share ? c->shard_member : -1, &t0, &t1);
    tp->prefix = c->d_prefix;
    tp->info = c->d_info;
    tp->T = c->T;
    if (share) {                 // the tensors that hold the share's first and last unit
        tp->u_lo = t1 > t0 ? tensor_of_unit(c, t0) : 0;
        tp->u_hi = t1 > t0 ? tensor_of_unit(c, t1 - 1) + 1 : 0;
    } else {
        tp->u_lo = bucket < 0 ? 0 : c->bucket_u_lo[bucket];
        tp->u_hi = bucket < 0 ? c->T : c->bucket_u_hi[bucket];
    }
    tp->tile_lo = t0;
    tp->n_tiles = t1 - t0;
    tp->tile = c->tile;
    tp->single = tp->u_hi - tp->u_lo == 1;
    tp->single_skip = 0;
    if (tp->single) {
        tp->one = c->info[tp->u_lo];
        tp->single_skip = t0 - c->prefix[tp->u_lo];
    }
    return KT_OK;
}

void bucket_range(const kt_ctx *c, int bucket, int64_t *lo, int64_t *n, bool whole = false) {
    if (sharded(c) && !whole) {
        int t0, t1;
        unit_range(c, bucket, c->shard_member, &t0, &t1);
        *lo = unit_start(c, t0);
        *n = unit_start(c, t1) - *lo;
        return;
    }
    if (bucket < 0) {
        *lo = 0;
        *n = c->transport_numel;
    } else {
        *lo = c->bucket_start[bucket];
        *n = c->bucket_numel[bucket];
    }
}

int check_ctx(const kt_ctx *c, bool need_plan) {
    if (!c) return fail(KT_ERR_INVALID, "ctx is NULL");
    if (need_plan && !c->planned) return fail(KT_ERR_STATE, "kt_bucket_pack has not been called on this context");
    return KT_OK;
}

int check_buffers(const kt_ctx *c, const float *const *bufs, int n, const char *what) {
    if (!bufs) return fail(KT_ERR_INVALID, "%s is NULL", what);
    for (int g = 0; g < n; ++g) {
        if (!bufs[g]) return fail(KT_ERR_INVALID, "%s[%d] is NULL", what, g);
        if (!aligned16(bufs[g])) return fail(KT_ERR_ALIGN, "%s[%d] is not 16-byte aligned", what, g);
    }
    (void)c;
    return KT_OK;
}

template <typename Tin>
int launch_k1(kt_ctx *c, const K1Params &p, cudaStream_t s) {
    // one CTA per tile; ranks are streamed in batches of KT_KB whatever K is: small batches keep
    // the register count at 64 and four CTAs resident per SM, which hides the tile look-up of
    // one CTA behind the loads of the others (measured: +12 % on ragged lists with K = 8)
    if (c->transport_dtype == KT_F32)
        k1_intra_reduce<Tin, float, KT_KB><<<p.tp.n_tiles, NT, 0, s>>>(p);
    else
        k1_intra_reduce<Tin, unsigned short, KT_KB><<<p.tp.n_tiles, NT, 0, s>>>(p);
    c->launches += 1;
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}

// combine + unpack: the tile size is the plan's (fixed by the gradient dtype), the vector
// width follows the output dtype, the loads the type of the source buffers
template <typename Tout, typename TT>
void launch_k2_typed(int tile, int n_tiles, cudaStream_t s, const K2Params &p) {
    if (tile == TILE_F32)
        k2_combine_unpack<Tout, TT, TILE_F32><<<n_tiles, NT, 0, s>>>(p);
    else
        k2_combine_unpack<Tout, TT, TILE_BF16><<<n_tiles, NT, 0, s>>>(p);
}

template <typename Tout>
void launch_k2(int tile, int n_tiles, cudaStream_t s, const K2Params &p, int src_dtype = KT_F32) {
    if (src_dtype == KT_F32) launch_k2_typed<Tout, float>(tile, n_tiles, s, p);
    else launch_k2_typed<Tout, unsigned short>(tile, n_tiles, s, p);
}

size_t transport_elem_size(const kt_ctx *c) { return c->transport_dtype == KT_F32 ? 4 : 2; }

int check_out_args(const kt_ctx *c, void *const *out_grads, int R, int out_dtype) {
    if (!out_grads) return fail(KT_ERR_INVALID, "out_grads is NULL");
    if (R < 1 || R > c->K) return fail(KT_ERR_SHAPE, "R = %d outside [1, K = %d]", R, c->K);
    if (out_dtype != KT_F32 && out_dtype != KT_BF16) return fail(KT_ERR_INVALID, "unknown out_dtype %d", out_dtype);
    const size_t es = out_dtype == KT_F32 ? 4 : 2;
    const int T = c->T;
    const size_t np = static_cast<size_t>(R) * T;
    for (size_t i = 0; i < np; ++i) {
        if (c->numel[i % T] > 0 && !out_grads[i]) return fail(KT_ERR_INVALID, "out_grads[%zu] is NULL", i);
        if (reinterpret_cast<uintptr_t>(out_grads[i]) % es) return fail(KT_ERR_ALIGN, "out_grads[%zu] is not element aligned", i);
    }
    return KT_OK;
}

// Destination table on the device: R*T pointers in transport tensor order, then one flag per
// tensor saying that all R destinations are 16-byte aligned.  Looked up among the context's
// sets; on a miss the least recently used set is replaced: its image is written into pinned
// host memory and uploaded with an asynchronous copy on the call's stream, after a stream-side
// wait for the last kernel that read the table it replaces.  Nothing here waits for the device
// unless a set has to grow or is replaced again while its own upload is still in flight.
// *set_out receives the set; the caller records set->used after its launch.
int upload_out_table(kt_ctx *c, void *const *out_grads, int R, int out_dtype, cudaStream_t s, bool capturing,
                     OutSet **set_out, size_t *sz_ptrs_out) {
    const int T = c->T;
    const size_t np = static_cast<size_t>(R) * T;
    const size_t sz_ptrs = round_up(np * sizeof(void *), 256);
    *sz_ptrs_out = sz_ptrs;
    OutSet *victim = nullptr;
    for (OutSet &o : c->out_sets) {
        if (o.dev && o.R == R && o.dtype == out_dtype && o.ptrs.size() == np &&
            std::memcmp(o.ptrs.data(), out_grads, np * sizeof(void *)) == 0) {
            o.stamp = ++c->out_clock;
            o.in_recording = o.in_recording || capturing;
            // the table was uploaded on another stream: this one must not run ahead of that copy
            // (while recording nothing is pending: kt_graph_begin has waited for every upload)
            if (!capturing && s != o.upload_stream) KT_CUDA(cudaStreamWaitEvent(s, o.uploaded, 0));
            *set_out = &o;
            return KT_OK;
        }
        if (!o.in_recording && (!victim || o.stamp < victim->stamp)) victim = &o;
    }
    if (capturing) {
        // an upload cannot be part of a recording: a replay would copy whatever the staging
        // image holds by then
        c->recording_broken = true;
        return fail(KT_ERR_STATE, "this set of output tensors is not on the device yet: run the step once "
                                  "with it before kt_graph_begin");
    }
    if (!victim)
        return fail(KT_ERR_STATE, "all %d destination tables of this context are held by recorded steps; "
                                  "kt_bucket_pack releases them", KT_OUT_SETS);
    OutSet &o = *victim;
    if (!o.uploaded) {
        KT_CUDA(cudaEventCreateWithFlags(&o.uploaded, cudaEventDisableTiming));
        KT_CUDA(cudaEventCreateWithFlags(&o.used, cudaEventDisableTiming));
    }
    const size_t need = sz_ptrs + round_up(T, 256);
    if (need > o.cap) {
        // kernels queued earlier may still read the old table: wait for the last of them, no more
        if (o.dev) {
            KT_CUDA(cudaEventSynchronize(o.used));
            KT_CUDA(cudaEventSynchronize(o.uploaded));
            cudaFree(o.dev);
            cudaFreeHost(o.staging);
            o.dev = nullptr;
            o.staging = nullptr;
            o.cap = 0;
            o.ptrs.clear();
        }
        if (cudaMalloc(&o.dev, need) != cudaSuccess) {
            cudaGetLastError();
            o.dev = nullptr;
            return fail(KT_ERR_NOMEM, "device allocation of %zu bytes failed", need);
        }
        if (cudaMallocHost(reinterpret_cast<void **>(&o.staging), need) != cudaSuccess) {
            cudaGetLastError();
            cudaFree(o.dev);
            o.dev = nullptr;
            o.staging = nullptr;
            return fail(KT_ERR_NOMEM, "pinned host allocation of %zu bytes failed", need);
        }
        o.cap = need;
    } else {
        KT_CUDA(cudaEventSynchronize(o.uploaded));       // the image may be rewritten only once it was read
        KT_CUDA(cudaStreamWaitEvent(s, o.used, 0));      // the table only once its last reader is done
    }
    o.ptrs.clear();                                      // not a valid set until the copy is queued
    std::memset(o.staging, 0, need);
    for (int cpy = 0; cpy < R; ++cpy)
        for (int u = 0; u < T; ++u)
            reinterpret_cast<void **>(o.staging)[static_cast<size_t>(cpy) * T + u] =
                out_grads[static_cast<size_t>(cpy) * T + (T - 1 - u)];
    for (int u = 0; u < T; ++u) {
        bool al = true;
        for (int cpy = 0; cpy < R; ++cpy) al = al && aligned16(out_grads[static_cast<size_t>(cpy) * T + (T - 1 - u)]);
        o.staging[sz_ptrs + u] = al ? 1 : 0;
    }
    KT_CUDA(cudaMemcpyAsync(o.dev, o.staging, need, cudaMemcpyHostToDevice, s));
    KT_CUDA(cudaEventRecord(o.uploaded, s));
    KT_CUDA(cudaEventRecord(o.used, s));
    o.upload_stream = s;
    o.ptrs.assign(out_grads, out_grads + np);
    o.R = R;
    o.dtype = out_dtype;
    o.stamp = ++c->out_clock;
    *set_out = &o;
    return KT_OK;
}

void forget_out_sets(kt_ctx *c) {
    // a new plan changes T and the tensor order: no uploaded table stays valid
    for (OutSet &o : c->out_sets) {
        o.ptrs.clear();
        o.R = 0;
        o.dtype = -1;
        o.in_recording = false;
    }
}

// A range of n elements cut into chunks of `chunk` elements (the last one shorter).
std::vector<int64_t> cut_chunks(int64_t n, int64_t chunk) {
    std::vector<int64_t> sizes;
    for (int64_t left = n; left > 0; left -= sizes.back()) sizes.push_back(left < chunk ? left : chunk);
    return sizes;
}

// Whether [p, p + bytes) lies inside ONE allocation (device memory, or host memory page-locked by
// one call).  Two allocations can be neighbours in the address space, yet a single copy must
// not run across the seam: the runtime rejects it.  Asked of the driver (start and size of the
// allocation that holds p); "no" whenever the driver cannot say.
bool one_allocation(const void *p, size_t bytes) {
    typedef CUresult (*attr_fn)(void *, CUpointer_attribute, CUdeviceptr);
    static const attr_fn query = [] {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult found;
        if (cudaGetDriverEntryPoint("cuPointerGetAttribute", &fn, cudaEnableDefault, &found) != cudaSuccess ||
            found != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            fn = nullptr;
        }
        return reinterpret_cast<attr_fn>(fn);
    }();
    if (!query) return false;
    const CUdeviceptr at = static_cast<CUdeviceptr>(reinterpret_cast<uintptr_t>(p));
    CUdeviceptr start = 0;
    size_t size = 0;
    if (query(&start, CU_POINTER_ATTRIBUTE_RANGE_START_ADDR, at) != CUDA_SUCCESS) return false;
    if (query(&size, CU_POINTER_ATTRIBUTE_RANGE_SIZE, at) != CUDA_SUCCESS) return false;
    return at >= start && bytes <= size && at - start <= size - bytes;
}

// One event per chunk of a relay ("chunk k went down: its way up may start"), created on demand.
int ensure_chunk_events(kt_ctx *c, size_t n_chunks) {
    while (c->chunk_events.size() < n_chunks) {
        cudaEvent_t e;
        KT_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        c->chunk_events.push_back(e);
    }
    return KT_OK;
}

bool is_capturing(cudaStream_t s) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &st) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return st != cudaStreamCaptureStatusNone;
}

}  // namespace

// ====================================================================== C ABI
extern "C" {

int kt_groups_init(const int32_t *group_of, const int32_t *shares, int K, int G, kt_ctx **out) {
    if (!out) return fail(KT_ERR_INVALID, "out is NULL");
    *out = nullptr;
    if (!group_of) return fail(KT_ERR_INVALID, "group_of is NULL");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (G < 1 || G > KT_MAX_GROUPS || G > K) return fail(KT_ERR_INVALID, "G = %d outside [1, min(K, %d)]", G, KT_MAX_GROUPS);
    if (int rc = check_shares(shares, K)) return rc;
    std::vector<int> members(G, 0);
    for (int r = 0; r < K; ++r) {
        if (group_of[r] < 0 || group_of[r] >= G) return fail(KT_ERR_INVALID, "group_of[%d] = %d outside [0, %d)", r, group_of[r], G);
        members[group_of[r]] += 1;
    }
    for (int g = 0; g < G; ++g)
        if (!members[g]) return fail(KT_ERR_INVALID, "group %d has no rank", g);

    kt_ctx *c = new (std::nothrow) kt_ctx();
    if (!c) return fail(KT_ERR_NOMEM, "out of host memory");
    c->K = K;
    c->G = G;
    c->group_of.assign(group_of, group_of + K);
    c->shares.assign(shares, shares + K);
    compute_coefficients(c);
    cudaError_t e = cudaGetDevice(&c->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_main, cudaEventDisableTiming);
    if (e != cudaSuccess) {
        delete c;
        return fail(KT_ERR_CUDA, "kt_groups_init: %s", cudaGetErrorString(e));
    }
    *out = c;
    return KT_OK;
}

int kt_set_shares(kt_ctx *c, const int32_t *shares) {
    if (int rc = check_ctx(c, false)) return rc;
    if (int rc = check_shares(shares, c->K)) return rc;
    c->shares.assign(shares, shares + c->K);
    return compute_coefficients(c);
}

int kt_set_coefficients(kt_ctx *c, const float *a, const float *W) {
    if (int rc = check_ctx(c, false)) return rc;
    if (!a || !W) return fail(KT_ERR_INVALID, "NULL argument");
    for (int k = 0; k < c->K; ++k) c->rt.coef[k] = a[c->order[k]];
    for (int g = 0; g < c->G; ++g) c->gt.W[g] = W[g];
    refresh_shard(c);
    return KT_OK;
}

int kt_set_transport_dtype(kt_ctx *c, int dtype) {
    if (int rc = check_ctx(c, false)) return rc;
    if (dtype != KT_F32 && dtype != KT_BF16) return fail(KT_ERR_INVALID, "unknown transport dtype %d", dtype);
    c->transport_dtype = dtype;
    return KT_OK;
}

int kt_get_coefficients(const kt_ctx *c, float *a_out, float *W_out) {
    if (int rc = check_ctx(c, false)) return rc;
    if (a_out)
        for (int k = 0; k < c->K; ++k) a_out[c->order[k]] = c->rt.coef[k];
    if (W_out)
        for (int g = 0; g < c->G; ++g) W_out[g] = c->gt.W[g];
    return KT_OK;
}

int kt_bucket_pack(kt_ctx *c, const void *const *grads, const int64_t *numel, int T, int in_dtype,
                   int64_t bucket_cap_bytes, void *const *flat_out, void *stream) {
    if (int rc = check_ctx(c, false)) return rc;
    if (!grads || !numel) return fail(KT_ERR_INVALID, "NULL argument");
    if (T < 1) return fail(KT_ERR_INVALID, "T = %d must be >= 1", T);
    if (in_dtype != KT_F32 && in_dtype != KT_BF16) return fail(KT_ERR_INVALID, "unknown in_dtype %d", in_dtype);
    if (bucket_cap_bytes < 4) return fail(KT_ERR_INVALID, "bucket_cap_bytes must be >= 4");
    const size_t es = in_dtype == KT_F32 ? 4 : 2;
    const int n_src = n_sources(c);
    if (flat_out && sharded(c))
        return fail(KT_ERR_STATE, "the standalone pack is not available on a context bound to one rank");
    for (int t = 0; t < T; ++t) {
        if (numel[t] < 0) return fail(KT_ERR_INVALID, "numel[%d] is negative", t);
        for (int r = 0; r < n_src; ++r) {
            const void *p = grads[static_cast<size_t>(r) * T + t];
            if (numel[t] > 0 && !p) return fail(KT_ERR_INVALID, "grads[%d][%d] is NULL", r, t);
            if (reinterpret_cast<uintptr_t>(p) % es) return fail(KT_ERR_ALIGN, "grads[%d][%d] is not element aligned", r, t);
        }
    }
    if (flat_out)
        for (int r = 0; r < c->K; ++r) {
            if (!flat_out[r]) return fail(KT_ERR_INVALID, "flat_out[%d] is NULL", r);
            if (!aligned16(flat_out[r])) return fail(KT_ERR_ALIGN, "flat_out[%d] is not 16-byte aligned", r);
        }

    BucketPlan bp;
    plan_buckets(numel, T, bucket_cap_bytes, &bp);
    const std::vector<int64_t> &offset = bp.offset;
    const std::vector<int32_t> &bof = bp.bucket_of;
    const std::vector<int64_t> &bstart = bp.start;
    const std::vector<int> &b_lo = bp.u_lo, &b_hi = bp.u_hi;
    const int64_t total = bp.total;
    const int nb = static_cast<int>(bstart.size());

    // ---- tile tables in transport order
    const int tile = in_dtype == KT_F32 ? TILE_F32 : TILE_BF16;
    std::vector<int> prefix(T + 1, 0);
    std::vector<TInfo> info(T);
    for (int u = 0; u < T; ++u) {
        const int t = T - 1 - u;
        const int64_t end = (u + 1 < T) ? offset[T - 2 - u] : total;
        TInfo &ti = info[u];
        ti.dst_off = offset[t];
        ti.numel = numel[t];
        ti.ext = end - offset[t];
        ti.flags = FLAG_ALIGNED;
        ti.pad_ = 0;
        for (int r = 0; r < n_src; ++r)
            if (!aligned16(grads[static_cast<size_t>(r) * T + t])) ti.flags = 0;
        const int64_t tiles = (ti.ext + tile - 1) / tile;
        if (prefix[u] + tiles > 0x7FFFFFF0LL) return fail(KT_ERR_SHAPE, "too many elements for one plan");
        prefix[u + 1] = prefix[u] + static_cast<int>(tiles);
    }
    std::vector<const void *> ptrs(static_cast<size_t>(n_src) * T);
    for (int k = 0; k < n_src; ++k)
        for (int u = 0; u < T; ++u)
            ptrs[static_cast<size_t>(k) * T + u] = grads[static_cast<size_t>(source_of(c, k)) * T + (T - 1 - u)];

    // ---- upload (one allocation, three 256-byte aligned regions)
    KT_ON_DEVICE(c->device);
    const size_t sz_prefix = round_up((T + 1) * sizeof(int), 256);
    const size_t sz_info = round_up(T * sizeof(TInfo), 256);
    const size_t sz_ptrs = round_up(ptrs.size() * sizeof(void *), 256);
    void *d = nullptr;
    if (cudaMalloc(&d, sz_prefix + sz_info + sz_ptrs) != cudaSuccess) {
        cudaGetLastError();
        return fail(KT_ERR_NOMEM, "device allocation of %zu bytes failed", sz_prefix + sz_info + sz_ptrs);
    }
    std::vector<char> staging(sz_prefix + sz_info + sz_ptrs, 0);
    std::memcpy(staging.data(), prefix.data(), (T + 1) * sizeof(int));
    std::memcpy(staging.data() + sz_prefix, info.data(), T * sizeof(TInfo));
    std::memcpy(staging.data() + sz_prefix + sz_info, ptrs.data(), ptrs.size() * sizeof(void *));
    cudaError_t e = cudaMemcpy(d, staging.data(), staging.size(), cudaMemcpyHostToDevice);
    if (e != cudaSuccess) {
        cudaFree(d);
        return fail(KT_ERR_CUDA, "table upload: %s", cudaGetErrorString(e));
    }
    if (c->d_tables) cudaFree(c->d_tables);
    c->d_tables = d;
    c->d_tables_bytes = sz_prefix + sz_info + sz_ptrs;
    c->d_prefix = static_cast<int *>(d);
    c->d_info = reinterpret_cast<TInfo *>(static_cast<char *>(d) + sz_prefix);
    c->d_ptrs = reinterpret_cast<const void **>(static_cast<char *>(d) + sz_prefix + sz_info);

    c->T = T;
    c->in_dtype = in_dtype;
    c->tile = tile;
    c->numel.assign(numel, numel + T);
    c->tensor_offset = offset;
    c->bucket_of = bof;
    c->bucket_start = bstart;
    c->bucket_numel.resize(nb);
    for (int b = 0; b < nb; ++b) c->bucket_numel[b] = (b + 1 < nb ? bstart[b + 1] : total) - bstart[b];
    c->bucket_u_lo = b_lo;
    c->bucket_u_hi = b_hi;
    c->transport_numel = total;
    c->prefix = prefix;
    c->info = info;
    c->planned = true;
    c->h_ptrs.assign(grads, grads + static_cast<size_t>(n_src) * T);
    forget_out_sets(c);
    for (int dir = 0; dir < 2; ++dir) {
        for (auto &s : c->slots[dir]) s.recorded = false;
        while (static_cast<int>(c->slots[dir].size()) < nb + 1) {
            StageSlot s;
            KT_CUDA(cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming));
            c->slots[dir].push_back(s);
        }
    }

    if (flat_out) {
        PackParams p{};
        if (int rc = make_tile_plan(c, -1, &p.tp)) return rc;
        p.ptrs = c->d_ptrs;
        p.K = c->K;
        for (int k = 0; k < c->K; ++k) p.flat[k] = flat_out[c->order[k]];
        if (p.tp.n_tiles > 0) {
            cudaStream_t s = static_cast<cudaStream_t>(stream);
            if (in_dtype == KT_F32)
                k_pack<float><<<dim3(p.tp.n_tiles, c->K), NT, 0, s>>>(p);
            else
                k_pack<unsigned short><<<dim3(p.tp.n_tiles, c->K), NT, 0, s>>>(p);
            c->launches += 1;
            KT_CUDA(cudaGetLastError());
        }
    }
    return KT_OK;
}

int kt_plan_query(const kt_ctx *c, int32_t *n_buckets, int64_t *bucket_start, int64_t *bucket_numel,
                  int64_t *tensor_offset, int32_t *bucket_of, int64_t *transport_numel) {
    if (int rc = check_ctx(c, true)) return rc;
    const int nb = static_cast<int>(c->bucket_start.size());
    if (n_buckets) *n_buckets = nb;
    if (bucket_start) std::memcpy(bucket_start, c->bucket_start.data(), nb * sizeof(int64_t));
    if (bucket_numel) std::memcpy(bucket_numel, c->bucket_numel.data(), nb * sizeof(int64_t));
    if (tensor_offset) std::memcpy(tensor_offset, c->tensor_offset.data(), c->T * sizeof(int64_t));
    if (bucket_of) std::memcpy(bucket_of, c->bucket_of.data(), c->T * sizeof(int32_t));
    if (transport_numel) *transport_numel = c->transport_numel;
    return KT_OK;
}

int kt_work_unit(int in_dtype) {
    if (in_dtype == KT_F32) return TILE_F32;
    if (in_dtype == KT_BF16) return TILE_BF16;
    return fail(KT_ERR_INVALID, "unknown dtype %d", in_dtype);
}

int kt_shard_bind(kt_ctx *c, int rank) {
    if (int rc = check_ctx(c, false)) return rc;
    if (rank < 0 || rank >= c->K) return fail(KT_ERR_INVALID, "rank = %d outside [0, %d)", rank, c->K);
    c->shard_rank = rank;
    c->shard_g = c->group_of[rank];
    c->shard_M = 0;
    for (int r = 0; r < c->K; ++r) {
        if (c->group_of[r] != c->shard_g) continue;
        if (r == rank) c->shard_member = c->shard_M;
        c->shard_M += 1;
    }
    refresh_shard(c);
    c->planned = false;          // the pointer table of an earlier plan had other rows
    return KT_OK;
}

int kt_shard_query(const kt_ctx *c, int bucket, int member, int *n_members, int64_t *lo, int64_t *n) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!sharded(c)) return fail(KT_ERR_STATE, "kt_shard_bind has not been called on this context");
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range [-1, %d)", bucket, (int)c->bucket_start.size());
    if (member < -1 || member >= c->shard_M) return fail(KT_ERR_INVALID, "member = %d outside [-1, %d)", member, c->shard_M);
    int t0, t1;
    unit_range(c, bucket, member < 0 ? c->shard_member : member, &t0, &t1);
    if (n_members) *n_members = c->shard_M;
    if (lo) *lo = unit_start(c, t0);
    if (n) *n = unit_start(c, t1) - unit_start(c, t0);
    return KT_OK;
}

int kt_hier_reduce(kt_ctx *c, int phase, int bucket, float *const *transport, float *combined, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (phase != KT_INTRA && phase != KT_INTER && phase != KT_BOTH) return fail(KT_ERR_INVALID, "unknown phase %d", phase);
    if (sharded(c) && phase == KT_INTRA) {       // only the own group's partial is written
        if (!transport) return fail(KT_ERR_INVALID, "transport is NULL");
        if (int rc = check_buffers(c, transport + c->shard_g, 1, "transport[own group]")) return rc;
    } else if (int rc = check_buffers(c, transport, c->G, "transport")) {
        return rc;
    }
    if (phase & KT_INTER) {
        if (!combined) return fail(KT_ERR_INVALID, "combined is NULL");
        if (!aligned16(combined)) return fail(KT_ERR_ALIGN, "combined is not 16-byte aligned");
    }
    TilePlan tp{};
    if (int rc = make_tile_plan(c, bucket, &tp)) return rc;
    KT_ON_DEVICE(c->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if ((phase & KT_INTRA) && tp.n_tiles > 0) {
        K1Params p{};
        p.tp = tp;
        p.ptrs = c->d_ptrs;
        p.rt = reduce_table(c);
        for (int g = 0; g < c->G; ++g) p.transport[g] = transport[g];
        p.wide = sharded(c) ? all_aligned32(transport + c->shard_g, 1) : all_aligned32(transport, c->G);
        const int rc = c->in_dtype == KT_F32 ? launch_k1<float>(c, p, s) : launch_k1<unsigned short>(c, p, s);
        if (rc) return rc;
    }
    if (phase & KT_INTER) {
        int64_t lo, n;
        bucket_range(c, bucket, &lo, &n);
        if (n > 0) {
            K2Params p{};
            p.gt = c->gt;
            for (int g = 0; g < c->G; ++g) p.src[g] = transport[g];
            const long long n4 = n / 4;   // bucket ranges are multiples of 64 elements
            if (c->transport_dtype == KT_F32)
                k_combine_flat<float><<<grid_for(c, k_combine_flat<float>, 0, (n4 + NT - 1) / NT), NT, 0, s>>>(p, combined, lo, n4);
            else
                k_combine_flat<unsigned short><<<grid_for(c, k_combine_flat<unsigned short>, 0, (n4 + NT - 1) / NT), NT, 0, s>>>(p, combined, lo, n4);
            c->launches += 1;
            KT_CUDA(cudaGetLastError());
        }
    }
    return KT_OK;
}

int kt_stage_to_host(kt_ctx *c, int dir, int bucket, float *const *transport, float *const *host_pinned,
                     void *main_stream, void *side_stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (dir != KT_D2H && dir != KT_H2D) return fail(KT_ERR_INVALID, "unknown direction %d", dir);
    if (!transport || !host_pinned) return fail(KT_ERR_INVALID, "NULL argument");
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range", bucket);
    // bound to one rank: the own group's partial goes down, the other groups' partials come up
    auto takes_part = [c, dir](int g) { return !sharded(c) || (dir == KT_D2H) == (g == c->shard_g); };
    for (int g = 0; g < c->G; ++g)
        if (takes_part(g) && (!transport[g] || !host_pinned[g])) return fail(KT_ERR_INVALID, "buffer %d is NULL", g);
    int64_t lo, n;
    bucket_range(c, bucket, &lo, &n);
    KT_ON_DEVICE(c->device);
    cudaStream_t ms = static_cast<cudaStream_t>(main_stream), ss = static_cast<cudaStream_t>(side_stream);
    KT_CUDA(cudaEventRecord(c->ev_main, ms));
    KT_CUDA(cudaStreamWaitEvent(ss, c->ev_main, 0));
    if (dir == KT_H2D) {
        // the way up reads what the way down wrote: wait for every copy down that covered any part
        // of this range -- the same bucket, the whole transport, and, when this call covers the
        // whole transport, every single bucket (they may have gone down on other streams)
        std::vector<StageSlot> &down = c->slots[KT_D2H];
        for (int i = 0; i < static_cast<int>(down.size()); ++i)
            if (down[i].recorded && (bucket < 0 || i == 0 || i == bucket + 1))
                KT_CUDA(cudaStreamWaitEvent(ss, down[i].done, 0));
    }
    const size_t es = transport_elem_size(c);
    for (int g = 0; g < c->G && n > 0; ++g) {
        if (!takes_part(g)) continue;
        char *dev = reinterpret_cast<char *>(transport[g]) + lo * es, *host = reinterpret_cast<char *>(host_pinned[g]) + lo * es;
        if (dir == KT_D2H)
            KT_CUDA(cudaMemcpyAsync(host, dev, n * es, cudaMemcpyDeviceToHost, ss));
        else
            KT_CUDA(cudaMemcpyAsync(dev, host, n * es, cudaMemcpyHostToDevice, ss));
    }
    StageSlot &slot = c->slots[dir][bucket + 1];
    KT_CUDA(cudaEventRecord(slot.done, ss));
    slot.recorded = true;
    return KT_OK;
}

int kt_relay_through_host(kt_ctx *c, int bucket, float *const *send, float *const *host_pinned,
                          float *const *recv, int64_t chunk_bytes, void *main_stream, void *d2h_stream,
                          void *h2d_stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!send || !host_pinned || !recv) return fail(KT_ERR_INVALID, "NULL argument");
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range", bucket);
    if (chunk_bytes < 256) return fail(KT_ERR_INVALID, "chunk_bytes must be >= 256");
    if (d2h_stream == h2d_stream) return fail(KT_ERR_INVALID, "the two copy streams must differ");
    if (sharded(c))
        return fail(KT_ERR_STATE, "bound to one rank, the way up reads what other processes copied down: use "
                                  "kt_stage_to_host per direction with a barrier between them");
    for (int g = 0; g < c->G; ++g)
        if (!send[g] || !host_pinned[g] || !recv[g]) return fail(KT_ERR_INVALID, "buffer %d is NULL", g);
    int64_t lo, n;
    bucket_range(c, bucket, &lo, &n);
    // When the whole transport moves and the G buffers of each set lie back to back in memory
    // (rows of one allocation), the relay treats them as one range: one copy per chunk and
    // direction instead of G, which matters because every copy costs the link a few microseconds.
    int groups = c->G;
    const size_t es = transport_elem_size(c);
    auto at_elem = [es](float *base, int64_t elem) { return reinterpret_cast<char *>(base) + elem * es; };
    if (bucket < 0) {
        bool rows = true;
        for (int g = 0; g + 1 < c->G; ++g)
            rows = rows && at_elem(send[g], n) == at_elem(send[g + 1], 0) &&
                   at_elem(host_pinned[g], n) == at_elem(host_pinned[g + 1], 0) &&
                   at_elem(recv[g], n) == at_elem(recv[g + 1], 0);
        // neighbours by address are not enough: each set must be one allocation, or a copy that
        // runs across the seam between two of them is refused
        const size_t all = static_cast<size_t>(n) * es * c->G;
        rows = rows && c->G > 1 && one_allocation(send[0], all) && one_allocation(host_pinned[0], all) &&
               one_allocation(recv[0], all);
        if (rows) {
            n *= c->G;
            groups = 1;
        }
    }
    // Uniform chunks (elements, a multiple of 64).  Shorter chunks at the two ends of the
    // pipeline were tried and measured slower: small copies use the host link badly.
    const std::vector<int64_t> sizes = cut_chunks(n, chunk_bytes / 256 * 256 / static_cast<int64_t>(es));
    const int64_t n_chunks = static_cast<int64_t>(sizes.size());
    KT_ON_DEVICE(c->device);
    if (int rc = ensure_chunk_events(c, sizes.size())) return rc;
    cudaStream_t ms = static_cast<cudaStream_t>(main_stream);
    cudaStream_t ds = static_cast<cudaStream_t>(d2h_stream), hs = static_cast<cudaStream_t>(h2d_stream);
    KT_CUDA(cudaEventRecord(c->ev_main, ms));
    KT_CUDA(cudaStreamWaitEvent(ds, c->ev_main, 0));
    KT_CUDA(cudaStreamWaitEvent(hs, c->ev_main, 0));
    int64_t at = lo;
    for (int64_t k = 0; k < n_chunks; at += sizes[k], ++k) {
        const size_t len = static_cast<size_t>(sizes[k]) * es;
        for (int g = 0; g < groups; ++g)
            KT_CUDA(cudaMemcpyAsync(at_elem(host_pinned[g], at), at_elem(send[g], at), len, cudaMemcpyDeviceToHost, ds));
        KT_CUDA(cudaEventRecord(c->chunk_events[k], ds));
        KT_CUDA(cudaStreamWaitEvent(hs, c->chunk_events[k], 0));
        for (int g = 0; g < groups; ++g)
            KT_CUDA(cudaMemcpyAsync(at_elem(recv[g], at), at_elem(host_pinned[g], at), len, cudaMemcpyHostToDevice, hs));
    }
    StageSlot &down = c->slots[KT_D2H][bucket + 1], &up = c->slots[KT_H2D][bucket + 1];
    KT_CUDA(cudaEventRecord(down.done, ds));
    down.recorded = true;
    KT_CUDA(cudaEventRecord(up.done, hs));
    up.recorded = true;
    return KT_OK;
}

int kt_stage_wait(kt_ctx *c, int dir, int bucket, void *main_stream, int timeout_ms) {
    if (int rc = check_ctx(c, true)) return rc;
    if (dir != KT_D2H && dir != KT_H2D) return fail(KT_ERR_INVALID, "unknown direction %d", dir);
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range", bucket);
    StageSlot &slot = c->slots[dir][bucket + 1];
    if (!slot.recorded) return fail(KT_ERR_STATE, "no staging copy queued for direction %d, bucket %d", dir, bucket);
    KT_CUDA(cudaStreamWaitEvent(static_cast<cudaStream_t>(main_stream), slot.done, 0));
    if (timeout_ms < 0) return KT_OK;
    // poll back to back for the first 300 us (a bucket's share crosses the link in about that
    // time), then with short sleeps, then with longer ones
    const auto begin = std::chrono::steady_clock::now();
    const auto deadline = begin + std::chrono::milliseconds(timeout_ms);
    for (;;) {
        const cudaError_t e = cudaEventQuery(slot.done);
        if (e == cudaSuccess) return KT_OK;
        if (e != cudaErrorNotReady) return fail(KT_ERR_CUDA, "cudaEventQuery: %s", cudaGetErrorString(e));
        const auto now = std::chrono::steady_clock::now();
        if (now >= deadline)
            return fail(KT_ERR_TIMEOUT, "staging copy (direction %d, bucket %d) not finished after %d ms", dir, bucket, timeout_ms);
        if (now - begin < std::chrono::microseconds(300)) continue;
        std::this_thread::sleep_for(std::chrono::microseconds(now - begin < std::chrono::milliseconds(5) ? 20 : 200));
    }
}

int kt_unpack_scale(kt_ctx *c, const float *const *src, int from_combined, void *const *out_grads, int R,
                    int out_dtype, float scale, int bucket, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    const int nsrc = from_combined ? 1 : c->G;
    if (int rc = check_out_args(c, out_grads, R, out_dtype)) return rc;
    if (int rc = check_buffers(c, src, nsrc, "src")) return rc;
    TilePlan tp{};
    if (int rc = make_tile_plan(c, bucket, &tp)) return rc;
    KT_ON_DEVICE(c->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    size_t sz_ptrs = 0;
    OutSet *set = nullptr;
    const bool capturing = is_capturing(s);
    if (int rc = upload_out_table(c, out_grads, R, out_dtype, s, capturing, &set, &sz_ptrs)) return rc;
    if (tp.n_tiles == 0) return KT_OK;

    K2Params p{};
    p.tp = tp;
    if (from_combined) {
        p.gt.G = 1;
        p.gt.W[0] = 1.0f;     // multiplying by one is exact: S passes through unchanged
        p.src[0] = src[0];
    } else {
        p.gt = c->gt;
        for (int g = 0; g < c->G; ++g) p.src[g] = src[g];
    }
    p.wide = all_aligned32(src, nsrc);
    p.out_ptrs = static_cast<void *const *>(set->dev);
    p.out_aligned = static_cast<const unsigned char *>(set->dev) + sz_ptrs;
    p.R = R;
    p.scale = scale;
    const int src_dtype = from_combined ? KT_F32 : c->transport_dtype;
    if (out_dtype == KT_F32)
        launch_k2<float>(tp.tile, tp.n_tiles, s, p, src_dtype);
    else
        launch_k2<unsigned short>(tp.tile, tp.n_tiles, s, p, src_dtype);
    c->launches += 1;
    KT_CUDA(cudaGetLastError());
    if (!capturing) KT_CUDA(cudaEventRecord(set->used, s));
    return KT_OK;
}

int kt_sync_direct(kt_ctx *c, void *const *out_grads, int R, int out_dtype, float scale, int bucket, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (sharded(c) && c->G > 1)
        return fail(KT_ERR_STATE, "bound to one rank, the one-pass route needs all ranks in one group (this context "
                                  "reads its own group's gradients only)");
    if (int rc = check_out_args(c, out_grads, R, out_dtype)) return rc;
    TilePlan tp{};
    if (int rc = make_tile_plan(c, bucket, &tp)) return rc;
    KT_ON_DEVICE(c->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    size_t sz_ptrs = 0;
    OutSet *set = nullptr;
    const bool capturing = is_capturing(s);
    if (int rc = upload_out_table(c, out_grads, R, out_dtype, s, capturing, &set, &sz_ptrs)) return rc;
    if (tp.n_tiles == 0) return KT_OK;

    DirectParams p{};
    p.tp = tp;
    p.ptrs = c->d_ptrs;
    p.rt = reduce_table(c);
    p.gt = c->gt;
    p.out_ptrs = static_cast<void *const *>(set->dev);
    p.out_aligned = static_cast<const unsigned char *>(set->dev) + sz_ptrs;
    p.R = R;
    p.scale = scale;
    // an output that is one of the registered gradient tensors (all-reduce in place, same element
    // type) is legal; the kernel then reads the gradients with ordinary loads
    bool inplace = false;
    if (c->in_dtype == out_dtype)
        for (int cpy = 0; cpy < R && !inplace; ++cpy)
            for (int t = 0; t < c->T && !inplace; ++t)
                for (int r = 0; r < n_sources(c) && !inplace; ++r)
                    inplace = c->numel[t] > 0 && out_grads[static_cast<size_t>(cpy) * c->T + t] ==
                                                     c->h_ptrs[static_cast<size_t>(r) * c->T + t];
    const bool in32 = c->in_dtype == KT_F32, out32 = out_dtype == KT_F32;
    if (in32 && out32) {
        if (inplace) k_direct_sync<float, float, KT_KB, true><<<tp.n_tiles, NT, 0, s>>>(p);
        else k_direct_sync<float, float, KT_KB, false><<<tp.n_tiles, NT, 0, s>>>(p);
    } else if (in32) {
        k_direct_sync<float, unsigned short, KT_KB, false><<<tp.n_tiles, NT, 0, s>>>(p);
    } else if (out32) {
        k_direct_sync<unsigned short, float, KT_KB_DIRECT_BF16, false><<<tp.n_tiles, NT, 0, s>>>(p);
    } else {
        if (inplace) k_direct_sync<unsigned short, unsigned short, KT_KB_DIRECT_BF16, true><<<tp.n_tiles, NT, 0, s>>>(p);
        else k_direct_sync<unsigned short, unsigned short, KT_KB_DIRECT_BF16, false><<<tp.n_tiles, NT, 0, s>>>(p);
    }
    c->launches += 1;
    KT_CUDA(cudaGetLastError());
    if (!capturing) KT_CUDA(cudaEventRecord(set->used, s));
    return KT_OK;
}

int kt_allreduce(kt_ctx *c, float *const *transport, float *const *host_pinned, float *const *recv,
                 void *const *out_grads, int R, int out_dtype, float scale, int64_t chunk_bytes, void *main_stream,
                 void *d2h_stream, void *h2d_stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (c->G == 1) return kt_sync_direct(c, out_grads, R, out_dtype, scale, -1, main_stream);
    if (sharded(c))
        return fail(KT_ERR_STATE, "bound to one rank, a collective that spans groups needs barriers between "
                                  "processes: call its parts (kt_hier_reduce, kt_stage_to_host, kt_unpack_scale)");
    if (int rc = check_out_args(c, out_grads, R, out_dtype)) return rc;      // fail before anything is queued
    if (int rc = kt_hier_reduce(c, KT_INTRA, -1, transport, nullptr, main_stream)) return rc;
    if (int rc = kt_relay_through_host(c, -1, transport, host_pinned, recv, chunk_bytes, main_stream, d2h_stream,
                                       h2d_stream))
        return rc;
    if (int rc = kt_stage_wait(c, KT_H2D, -1, main_stream, -1)) return rc;
    return kt_unpack_scale(c, recv, 0, out_grads, R, out_dtype, scale, -1, main_stream);
}

int kt_cast(const void *in, int in_dtype, void *out, int out_dtype, int64_t n, void *stream) {
    if (n < 0) return fail(KT_ERR_INVALID, "n is negative");
    if (n == 0) return KT_OK;
    if (!in || !out) return fail(KT_ERR_INVALID, "NULL argument");
    if ((in_dtype != KT_F32 && in_dtype != KT_BF16) || (out_dtype != KT_F32 && out_dtype != KT_BF16))
        return fail(KT_ERR_INVALID, "unknown dtype");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (in_dtype == out_dtype) {
        KT_CUDA(cudaMemcpyAsync(out, in, n * (in_dtype == KT_F32 ? 4 : 2), cudaMemcpyDeviceToDevice, s));
        return KT_OK;
    }
    int dev = 0, sms = 0;
    KT_CUDA(cudaGetDevice(&dev));
    KT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    long long blocks = (n + NT - 1) / NT;
    const long long cap = static_cast<long long>(sms) * 8;
    const int grid = static_cast<int>(blocks < cap ? blocks : cap);
    if (in_dtype == KT_BF16)
        k_cast_bf16_to_f32<<<grid, NT, 0, s>>>(static_cast<const unsigned short *>(in), static_cast<float *>(out), n);
    else
        k_cast_f32_to_bf16<<<grid, NT, 0, s>>>(static_cast<const float *>(in), static_cast<unsigned short *>(out), n);
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}

int kt_copy_tensors(void *const *dst, const void *const *src, const int64_t *bytes, int n, int dir, void *stream) {
    if (n < 0) return fail(KT_ERR_INVALID, "n is negative");
    if (n == 0) return KT_OK;
    if (!dst || !src || !bytes) return fail(KT_ERR_INVALID, "NULL argument");
    if (dir != KT_D2H && dir != KT_H2D) return fail(KT_ERR_INVALID, "unknown direction %d", dir);
    const cudaMemcpyKind kind = dir == KT_D2H ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < n; ++i) {
        if (bytes[i] < 0) return fail(KT_ERR_INVALID, "bytes[%d] is negative", i);
        if (bytes[i] > 0 && (!dst[i] || !src[i])) return fail(KT_ERR_INVALID, "pointer %d is NULL", i);
    }
    // one copy per tensor: neighbouring tensors may belong to different host registrations,
    // which a single copy must not span
    for (int i = 0; i < n; ++i)
        if (bytes[i] > 0) KT_CUDA(cudaMemcpyAsync(dst[i], src[i], static_cast<size_t>(bytes[i]), kind, s));
    return KT_OK;
}

// ---- memory shared between the processes of one node
namespace {
struct IpcEntry {
    unsigned char handle[KT_IPC_HANDLE_BYTES];
    int device;
    void *base;
    int refs;
};
std::mutex g_ipc_mutex;
std::vector<IpcEntry> g_ipc_open;      // every handle is opened once per process and device, then counted
}  // namespace

int kt_ipc_export(const void *dev_ptr, void *handle_out, int64_t *offset_out) {
    if (!dev_ptr || !handle_out || !offset_out) return fail(KT_ERR_INVALID, "NULL argument");
    static_assert(sizeof(cudaIpcMemHandle_t) == KT_IPC_HANDLE_BYTES, "handle size");
    // the handle names the whole allocation; where inside it the pointer lies is asked of the driver
    typedef int (*range_fn)(unsigned long long *, size_t *, unsigned long long);
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult found;
    KT_CUDA(cudaGetDriverEntryPoint("cuMemGetAddressRange", &fn, cudaEnableDefault, &found));
    if (!fn || found != cudaDriverEntryPointSuccess) return fail(KT_ERR_CUDA, "the driver does not offer cuMemGetAddressRange");
    unsigned long long base = 0;
    size_t size = 0;
    const int drc = reinterpret_cast<range_fn>(fn)(&base, &size, static_cast<unsigned long long>(reinterpret_cast<uintptr_t>(dev_ptr)));
    if (drc != 0) return fail(KT_ERR_CUDA, "cuMemGetAddressRange failed with driver status %d (not a device allocation?)", drc);
    cudaIpcMemHandle_t h;
    KT_CUDA(cudaIpcGetMemHandle(&h, reinterpret_cast<void *>(static_cast<uintptr_t>(base))));
    std::memcpy(handle_out, &h, sizeof(h));
    *offset_out = static_cast<int64_t>(reinterpret_cast<uintptr_t>(dev_ptr) - base);
    return KT_OK;
}

int kt_ipc_open(const void *handle, int64_t offset, void **dev_ptr_out) {
    if (!handle || !dev_ptr_out) return fail(KT_ERR_INVALID, "NULL argument");
    if (offset < 0) return fail(KT_ERR_INVALID, "offset is negative");
    int dev = 0;
    KT_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_ipc_mutex);
    for (IpcEntry &e : g_ipc_open)
        if (e.device == dev && std::memcmp(e.handle, handle, KT_IPC_HANDLE_BYTES) == 0) {
            e.refs += 1;
            *dev_ptr_out = static_cast<char *>(e.base) + offset;
            return KT_OK;
        }
    cudaIpcMemHandle_t h;
    std::memcpy(&h, handle, sizeof(h));
    void *base = nullptr;
    KT_CUDA(cudaIpcOpenMemHandle(&base, h, cudaIpcMemLazyEnablePeerAccess));
    IpcEntry e;
    std::memcpy(e.handle, handle, KT_IPC_HANDLE_BYTES);
    e.device = dev;
    e.base = base;
    e.refs = 1;
    g_ipc_open.push_back(e);
    *dev_ptr_out = static_cast<char *>(base) + offset;
    return KT_OK;
}

int kt_ipc_close(const void *handle) {
    if (!handle) return fail(KT_ERR_INVALID, "NULL argument");
    int dev = 0;
    KT_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lock(g_ipc_mutex);
    for (size_t i = 0; i < g_ipc_open.size(); ++i) {
        IpcEntry &e = g_ipc_open[i];
        if (e.device != dev || std::memcmp(e.handle, handle, KT_IPC_HANDLE_BYTES) != 0) continue;
        if (--e.refs == 0) {
            void *base = e.base;
            g_ipc_open.erase(g_ipc_open.begin() + static_cast<long>(i));
            KT_CUDA(cudaIpcCloseMemHandle(base));
        }
        return KT_OK;
    }
    return fail(KT_ERR_STATE, "this handle is not open on device %d", dev);
}

int kt_host_register(void *host, int64_t bytes) {
    if (!host || bytes < 1) return fail(KT_ERR_INVALID, "bad host range");
    KT_CUDA(cudaHostRegister(host, static_cast<size_t>(bytes), cudaHostRegisterPortable));
    return KT_OK;
}

int kt_host_unregister(void *host) {
    if (!host) return fail(KT_ERR_INVALID, "NULL argument");
    KT_CUDA(cudaHostUnregister(host));
    return KT_OK;
}

int kt_shard_step(kt_ctx *c, void *barrier_block, float *const *partials, float *const *host_shared,
                  void *const *out_grads, int R, int out_dtype, float scale, int per_bucket, void *main_stream,
                  void *down_stream, void *up_stream, int timeout_ms) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!sharded(c)) return fail(KT_ERR_STATE, "kt_shard_bind has not been called on this context");
    if (!barrier_block) return fail(KT_ERR_INVALID, "barrier_block is NULL");
    if (c->G > 1 && (!partials || !host_shared)) return fail(KT_ERR_INVALID, "partials and host_shared are needed with several groups");
    if (c->G > 1 && down_stream == up_stream) return fail(KT_ERR_INVALID, "the two copy streams must differ");
    if (int rc = check_out_args(c, out_grads, R, out_dtype)) return rc;          // fail before the first barrier
    const int nb = static_cast<int>(c->bucket_start.size());
    const int first = per_bucket ? 0 : -1, past = per_bucket ? nb : 0;
    cudaStream_t ms = static_cast<cudaStream_t>(main_stream);
    {
        KT_ON_DEVICE(c->device);
        KT_CUDA(cudaDeviceSynchronize());                  // whatever produced this rank's gradients is done
    }
    if (int rc = kt_host_barrier(barrier_block, c->K, timeout_ms)) return rc;    // ... and so is everybody's
    if (c->G == 1) {
        for (int b = first; b < past; ++b)
            if (int rc = kt_sync_direct(c, out_grads, R, out_dtype, scale, b, main_stream)) return rc;
    } else {
        // all reduces are queued at once; the shares go down range by range behind them
        for (int b = first; b < past; ++b) {
            if (int rc = kt_hier_reduce(c, KT_INTRA, b, partials, nullptr, main_stream)) return rc;
            if (int rc = kt_stage_to_host(c, KT_D2H, b, partials, host_shared, main_stream, down_stream)) return rc;
        }
        // range by range: once every rank's share of a range is in host memory its way up starts,
        // on the other copy stream, while the later ranges are still on their way down
        for (int b = first; b < past; ++b) {
            // a wait without limit would hide a dead device behind a dead rank: the copy gets the same limit
            if (int rc = kt_stage_wait(c, KT_D2H, b, main_stream, timeout_ms < 0 ? 3600 * 1000 : timeout_ms)) return rc;
            if (int rc = kt_host_barrier(barrier_block, c->K, timeout_ms)) return rc;
            if (int rc = kt_stage_to_host(c, KT_H2D, b, partials, host_shared, main_stream, up_stream)) return rc;
            if (int rc = kt_stage_wait(c, KT_H2D, b, main_stream, -1)) return rc;
            if (int rc = kt_unpack_scale(c, partials, 0, out_grads, R, out_dtype, scale, b, main_stream)) return rc;
        }
    }
    {
        KT_ON_DEVICE(c->device);
        KT_CUDA(cudaStreamSynchronize(ms));                // this rank's shares are written everywhere in its group
    }
    return kt_host_barrier(barrier_block, c->K, timeout_ms);
}

int kt_shard_bcast(kt_ctx *c, int root, void *barrier_block, void *send, void *host_shared, void *recv,
                   int per_bucket, void *main_stream, void *d2h_stream, void *h2d_stream, int timeout_ms) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!sharded(c)) return fail(KT_ERR_STATE, "kt_shard_bind has not been called on this context");
    if (root < 0 || root >= c->K) return fail(KT_ERR_INVALID, "root = %d outside [0, %d)", root, c->K);
    if (!barrier_block) return fail(KT_ERR_INVALID, "barrier_block is NULL");
    const bool is_root = c->shard_rank == root, roots_group = c->group_of[root] == c->shard_g;
    if (is_root && !send) return fail(KT_ERR_INVALID, "send is NULL");
    if (c->G > 1 && !host_shared) return fail(KT_ERR_INVALID, "host_shared is NULL");
    if (!roots_group && !recv) return fail(KT_ERR_INVALID, "recv is NULL");
    const int nb = static_cast<int>(c->bucket_start.size());
    const int first = per_bucket ? 0 : -1, past = per_bucket ? nb : 0;
    const int64_t chunk = int64_t(1) << 40;                  // each half is one copy per range
    void *recv_rows[KT_MAX_GROUPS] = {};
    recv_rows[c->shard_g] = recv;
    {
        KT_ON_DEVICE(c->device);
        KT_CUDA(cudaDeviceSynchronize());                     // nothing on this device still touches the tensors
    }
    if (int rc = kt_host_barrier(barrier_block, c->K, timeout_ms)) return rc;
    if (is_root) {
        for (int b = first; b < past; ++b) {
            if (int rc = kt_bcast_send(c, root, b, send, main_stream)) return rc;
            if (c->G > 1)
                if (int rc = kt_bcast_relay(c, root, b, send, host_shared, recv_rows, chunk, main_stream, d2h_stream, h2d_stream))
                    return rc;
        }
        if (c->G > 1)
            for (int b = first; b < past; ++b)
                if (int rc = kt_stage_wait(c, KT_D2H, b, main_stream, timeout_ms < 0 ? 3600 * 1000 : timeout_ms)) return rc;
    }
    if (int rc = kt_host_barrier(barrier_block, c->K, timeout_ms)) return rc;   // the root's tensors are in host memory
    if (!roots_group) {
        for (int b = first; b < past; ++b)
            if (int rc = kt_bcast_relay(c, root, b, nullptr, host_shared, recv_rows, chunk, main_stream, d2h_stream, h2d_stream))
                return rc;
        for (int b = first; b < past; ++b) {
            if (int rc = kt_stage_wait(c, KT_H2D, b, main_stream, -1)) return rc;
            if (int rc = kt_bcast_recv(c, root, b, recv_rows, main_stream)) return rc;
        }
    }
    {
        KT_ON_DEVICE(c->device);
        KT_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(main_stream)));
    }
    return kt_host_barrier(barrier_block, c->K, timeout_ms);
}

int64_t kt_launch_count(const kt_ctx *c) { return c ? c->launches : 0; }

void kt_destroy(kt_ctx *c) {
    if (!c) return;
    DeviceScope device_scope_(c->device);
    bool tables = c->d_tables != nullptr;
    for (const OutSet &o : c->out_sets) tables = tables || o.dev;
    if (tables) cudaDeviceSynchronize();
    if (c->d_tables) cudaFree(c->d_tables);
    for (OutSet &o : c->out_sets) {
        if (o.dev) cudaFree(o.dev);
        if (o.staging) cudaFreeHost(o.staging);
        if (o.uploaded) cudaEventDestroy(o.uploaded);
        if (o.used) cudaEventDestroy(o.used);
    }
    if (c->ev_main) cudaEventDestroy(c->ev_main);
    for (int dir = 0; dir < 2; ++dir)
        for (auto &s : c->slots[dir])
            if (s.done) cudaEventDestroy(s.done);
    for (cudaEvent_t e : c->chunk_events) cudaEventDestroy(e);
    delete c;
}

}  // extern "C"

// ---------------------------------------------------------------------- one-submission step (CUDA graph)
struct kt_graph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    int device = 0;
    size_t nodes = 0;
};

extern "C" {

int kt_graph_begin(kt_ctx *c, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    KT_ON_DEVICE(c->device);
    // destination tables uploaded by earlier calls must be complete before a recording relies on
    // them: a recorded launch cannot wait for an event from outside the recording
    for (OutSet &o : c->out_sets)
        if (o.uploaded) KT_CUDA(cudaEventSynchronize(o.uploaded));
    // thread-local mode: other threads of the process may keep allocating while this one records
    KT_CUDA(cudaStreamBeginCapture(static_cast<cudaStream_t>(stream), cudaStreamCaptureModeThreadLocal));
    c->recording_broken = false;
    return KT_OK;
}

int kt_graph_end(kt_ctx *c, void *stream, kt_graph **out) {
    if (!out) return fail(KT_ERR_INVALID, "out is NULL");
    *out = nullptr;
    if (int rc = check_ctx(c, true)) return rc;
    cudaGraph_t g = nullptr;
    cudaError_t e = cudaStreamEndCapture(static_cast<cudaStream_t>(stream), &g);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(KT_ERR_CUDA, "cudaStreamEndCapture: %s (a copy stream that was not waited for, or a call "
                                 "that cannot be recorded, ends a recording this way)", cudaGetErrorString(e));
    }
    if (c->recording_broken) {
        c->recording_broken = false;
        if (g) cudaGraphDestroy(g);
        return fail(KT_ERR_STATE, "a call made while recording was refused (it needed an upload or an allocation): "
                                  "the recording is incomplete and was dropped");
    }
    kt_graph *h = new (std::nothrow) kt_graph();
    if (!h) {
        cudaGraphDestroy(g);
        return fail(KT_ERR_NOMEM, "out of host memory");
    }
    h->graph = g;
    h->device = c->device;
    cudaGraphGetNodes(g, nullptr, &h->nodes);
    e = cudaGraphInstantiate(&h->exec, g, 0);
    if (e != cudaSuccess) {
        cudaGraphDestroy(g);
        delete h;
        return fail(KT_ERR_CUDA, "cudaGraphInstantiate: %s", cudaGetErrorString(e));
    }
    *out = h;
    return KT_OK;
}

int kt_graph_launch(kt_graph *g, void *stream) {
    if (!g || !g->exec) return fail(KT_ERR_INVALID, "graph is NULL");
    KT_CUDA(cudaGraphLaunch(g->exec, static_cast<cudaStream_t>(stream)));
    return KT_OK;
}

int64_t kt_graph_nodes(const kt_graph *g) { return g ? static_cast<int64_t>(g->nodes) : 0; }

void kt_graph_destroy(kt_graph *g) {
    if (!g) return;
    if (g->exec) cudaGraphExecDestroy(g->exec);
    if (g->graph) cudaGraphDestroy(g->graph);
    delete g;
}

}  // extern "C"

// ---------------------------------------------------------------------- load-adaptive sampler (index kernel)
extern "C" {

int kt_sampler_indices(const int64_t *list, int64_t dataset_size, const int32_t *shares, int K, int drop_last,
                       int64_t *const *out, void *stream) {
    if (!out) return fail(KT_ERR_INVALID, "out is NULL");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (int rc = check_shares(shares, K)) return rc;
    if (dataset_size < 1) return fail(KT_ERR_INVALID, "dataset_size must be >= 1");
    SamplerParams p{};
    long long B = 0;
    for (int r = 0; r < K; ++r) {
        p.start[r] = static_cast<int>(B);
        B += shares[r];
        if (B > 0x7FFFFFFFLL) return fail(KT_ERR_SHAPE, "global batch too large");
    }
    p.start[K] = static_cast<int>(B);
    const int64_t steps = kt_sampler_steps(dataset_size, B, drop_last);
    if (steps == 0) return KT_OK;
    for (int r = 0; r < K; ++r) {
        if (!out[r]) return fail(KT_ERR_INVALID, "out[%d] is NULL", r);
        if (reinterpret_cast<uintptr_t>(out[r]) % 8) return fail(KT_ERR_ALIGN, "out[%d] is not 8-byte aligned", r);
        p.out[r] = reinterpret_cast<long long *>(out[r]);
    }
    if (reinterpret_cast<uintptr_t>(list) % 8) return fail(KT_ERR_ALIGN, "list is not 8-byte aligned");
    p.list = reinterpret_cast<const long long *>(list);
    p.D = dataset_size;
    p.B = static_cast<int>(B);
    p.K = K;
    p.total = steps * B;
    int dev = 0, sms = 0;
    KT_CUDA(cudaGetDevice(&dev));
    KT_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const long long blocks = (p.total + NT - 1) / NT, cap = static_cast<long long>(sms) * 8;
    k_sampler<<<static_cast<int>(blocks < cap ? blocks : cap), NT, 0, static_cast<cudaStream_t>(stream)>>>(p);
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------- hierarchical broadcast
namespace {

int fill_bcast(const kt_ctx *c, int root, BcastParams *p) {
    if (root < 0 || root >= c->K) return fail(KT_ERR_INVALID, "root = %d outside [0, %d)", root, c->K);
    p->ptrs = const_cast<void *const *>(reinterpret_cast<const void *const *>(c->d_ptrs));
    if (sharded(c)) {
        // The pointer table holds the M members of this rank's group only.  The kernels see two
        // "groups": 0 is the root's side (the members, when this rank's group is the root's; empty
        // otherwise), 1 the receiving side (the members, when it is not).
        p->G = 2;
        p->g_root = 0;
        p->k_root = 0;
        const bool roots_group = c->group_of[root] == c->shard_g;
        p->k_lo[0] = 0;
        p->k_hi[0] = static_cast<unsigned char>(roots_group ? c->shard_M : 0);
        p->k_lo[1] = 0;
        p->k_hi[1] = static_cast<unsigned char>(roots_group ? 0 : c->shard_M);
        if (roots_group)
            for (int r = 0, m = 0; r < c->K; ++r) {
                if (c->group_of[r] != c->shard_g) continue;
                if (r == root) p->k_root = m;
                ++m;
            }
        return KT_OK;
    }
    p->G = c->G;
    p->g_root = c->group_of[root];
    for (int g = 0; g < c->G; ++g) p->k_lo[g] = p->k_hi[g] = 0;
    for (int k = 0; k < c->K; ++k) {
        const int g = c->group_of[c->order[k]];
        if (k == 0 || c->group_of[c->order[k - 1]] != g) p->k_lo[g] = static_cast<unsigned char>(k);
        p->k_hi[g] = static_cast<unsigned char>(k + 1);
        if (c->order[k] == root) p->k_root = k;
    }
    return KT_OK;
}

}  // namespace

extern "C" {

int kt_bcast_send(kt_ctx *c, int root, int bucket, void *send, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!send) return fail(KT_ERR_INVALID, "send is NULL");
    if (!aligned16(send)) return fail(KT_ERR_ALIGN, "send is not 16-byte aligned");
    BcastParams p{};
    if (int rc = fill_bcast(c, root, &p)) return rc;
    if (sharded(c) && c->shard_rank != root) return KT_OK;      // only the root's own device sends
    if (int rc = make_tile_plan(c, bucket, &p.tp, true)) return rc;
    if (p.tp.n_tiles == 0) return KT_OK;
    p.flat[p.g_root] = send;
    KT_ON_DEVICE(c->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c->in_dtype == KT_F32) k_bcast_send<float><<<p.tp.n_tiles, NT, 0, s>>>(p);
    else k_bcast_send<unsigned short><<<p.tp.n_tiles, NT, 0, s>>>(p);
    c->launches += 1;
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}

int kt_bcast_recv(kt_ctx *c, int root, int bucket, void *const *recv, void *stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!recv) return fail(KT_ERR_INVALID, "recv is NULL");
    BcastParams p{};
    if (int rc = fill_bcast(c, root, &p)) return rc;
    if (sharded(c)) {
        // a rank of another group unpacks its share of its group's receive buffer into the tensors
        // of every member; the ranks of the root's group were written by the root itself
        if (c->group_of[root] == c->shard_g) return KT_OK;
        void *mine = recv[c->shard_g];
        if (!mine) return fail(KT_ERR_INVALID, "recv[%d] is NULL", c->shard_g);
        if (!aligned16(mine)) return fail(KT_ERR_ALIGN, "recv[%d] is not 16-byte aligned", c->shard_g);
        p.flat[1] = mine;
    } else {
        for (int g = 0; g < c->G; ++g) {
            if (g == p.g_root) continue;
            if (!recv[g]) return fail(KT_ERR_INVALID, "recv[%d] is NULL", g);
            if (!aligned16(recv[g])) return fail(KT_ERR_ALIGN, "recv[%d] is not 16-byte aligned", g);
            p.flat[g] = recv[g];
        }
    }
    if (int rc = make_tile_plan(c, bucket, &p.tp)) return rc;
    if (p.tp.n_tiles == 0 || c->G == 1) return KT_OK;
    KT_ON_DEVICE(c->device);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c->in_dtype == KT_F32) k_bcast_recv<float><<<p.tp.n_tiles, NT, 0, s>>>(p);
    else k_bcast_recv<unsigned short><<<p.tp.n_tiles, NT, 0, s>>>(p);
    c->launches += 1;
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}

int kt_bcast_relay(kt_ctx *c, int root, int bucket, const void *send, void *host_pinned, void *const *recv,
                   int64_t chunk_bytes, void *main_stream, void *d2h_stream, void *h2d_stream) {
    if (int rc = check_ctx(c, true)) return rc;
    if (!host_pinned) return fail(KT_ERR_INVALID, "host_pinned is NULL");
    if (root < 0 || root >= c->K) return fail(KT_ERR_INVALID, "root = %d outside [0, %d)", root, c->K);
    if (bucket < -1 || bucket >= static_cast<int>(c->bucket_start.size()))
        return fail(KT_ERR_SHAPE, "bucket %d out of range", bucket);
    if (chunk_bytes < 256) return fail(KT_ERR_INVALID, "chunk_bytes must be >= 256");
    if (d2h_stream == h2d_stream) return fail(KT_ERR_INVALID, "the two copy streams must differ");
    if (sharded(c)) {
        // One half per role, the caller's barrier between them: the root copies the whole range
        // down; a rank of another group copies its share up; the root's group mates do nothing.
        const bool is_root = c->shard_rank == root, roots_group = c->group_of[root] == c->shard_g;
        if (!is_root && roots_group) return KT_OK;
        if (is_root && !send) return fail(KT_ERR_INVALID, "send is NULL");
        if (!is_root && (!recv || !recv[c->shard_g])) return fail(KT_ERR_INVALID, "recv[%d] is NULL", c->shard_g);
        int64_t lo, n;
        bucket_range(c, bucket, &lo, &n, is_root);
        const size_t es = c->in_dtype == KT_F32 ? 4 : 2;
        KT_ON_DEVICE(c->device);
        cudaStream_t ms = static_cast<cudaStream_t>(main_stream);
        cudaStream_t cs = static_cast<cudaStream_t>(is_root ? d2h_stream : h2d_stream);
        KT_CUDA(cudaEventRecord(c->ev_main, ms));
        KT_CUDA(cudaStreamWaitEvent(cs, c->ev_main, 0));
        char *host = static_cast<char *>(host_pinned) + static_cast<size_t>(lo) * es;
        if (n > 0) {
            if (is_root)
                KT_CUDA(cudaMemcpyAsync(host, static_cast<const char *>(send) + static_cast<size_t>(lo) * es,
                                        static_cast<size_t>(n) * es, cudaMemcpyDeviceToHost, cs));
            else
                KT_CUDA(cudaMemcpyAsync(static_cast<char *>(recv[c->shard_g]) + static_cast<size_t>(lo) * es, host,
                                        static_cast<size_t>(n) * es, cudaMemcpyHostToDevice, cs));
        }
        StageSlot &slot = c->slots[is_root ? KT_D2H : KT_H2D][bucket + 1];
        KT_CUDA(cudaEventRecord(slot.done, cs));
        slot.recorded = true;
        return KT_OK;
    }
    if (!send || !recv) return fail(KT_ERR_INVALID, "NULL argument");
    const int g_root = c->group_of[root];
    for (int g = 0; g < c->G; ++g)
        if (g != g_root && !recv[g]) return fail(KT_ERR_INVALID, "recv[%d] is NULL", g);
    int64_t lo, n;
    bucket_range(c, bucket, &lo, &n);
    const size_t es = c->in_dtype == KT_F32 ? 4 : 2;
    const std::vector<int64_t> sizes = cut_chunks(n, chunk_bytes / 256 * 256 / static_cast<int64_t>(es));
    const int64_t n_chunks = static_cast<int64_t>(sizes.size());
    KT_ON_DEVICE(c->device);
    if (int rc = ensure_chunk_events(c, sizes.size())) return rc;
    cudaStream_t ms = static_cast<cudaStream_t>(main_stream);
    cudaStream_t ds = static_cast<cudaStream_t>(d2h_stream), hs = static_cast<cudaStream_t>(h2d_stream);
    KT_CUDA(cudaEventRecord(c->ev_main, ms));
    KT_CUDA(cudaStreamWaitEvent(ds, c->ev_main, 0));
    KT_CUDA(cudaStreamWaitEvent(hs, c->ev_main, 0));
    const char *src = static_cast<const char *>(send);
    char *host = static_cast<char *>(host_pinned);
    int64_t at = lo;
    for (int64_t k = 0; k < n_chunks; at += sizes[k], ++k) {
        const size_t off = static_cast<size_t>(at) * es, len = static_cast<size_t>(sizes[k]) * es;
        KT_CUDA(cudaMemcpyAsync(host + off, src + off, len, cudaMemcpyDeviceToHost, ds));
        KT_CUDA(cudaEventRecord(c->chunk_events[k], ds));
        KT_CUDA(cudaStreamWaitEvent(hs, c->chunk_events[k], 0));
        for (int g = 0; g < c->G; ++g)
            if (g != g_root)
                KT_CUDA(cudaMemcpyAsync(static_cast<char *>(recv[g]) + off, host + off, len, cudaMemcpyHostToDevice, hs));
    }
    StageSlot &down = c->slots[KT_D2H][bucket + 1], &up = c->slots[KT_H2D][bucket + 1];
    KT_CUDA(cudaEventRecord(down.done, ds));
    down.recorded = true;
    KT_CUDA(cudaEventRecord(up.done, hs));
    up.recorded = true;
    return KT_OK;
}

}  // extern "C"

// ====================================================================== entry point that allocates nothing
// For callers that must not allocate: code running where cudaMalloc is off limits (inside a
// region that forbids synchronising allocations, under a memory pool it may not touch, late
// in a process whose device memory is spoken for).  The whole flat path -- weighted
// intra-group reduce, combine, scale, cast -- runs with its scratch (tensor table, pointer
// tables and the fp32 group partials) in one file-scope device array of fixed size.
namespace {

constexpr size_t STATIC_TABLE_BYTES = 4096;

struct StaticTables {                   // image of the first bytes of the scratch
    int prefix[8];                      // tiles before tensor 0 and 1
    TInfo info;                         // the one tensor
    const void *in_ptrs[KT_MAX_RANKS];
    void *out_ptr[1];
    unsigned char out_aligned[8];
};
static_assert(sizeof(StaticTables) <= STATIC_TABLE_BYTES, "tables outgrew their slot");
static_assert(sizeof(StaticTables) % 16 == 0 && offsetof(StaticTables, info) % 16 == 0,
              "the tables are written, and the tensor record read, in 16-byte words");

// Held by every GPU that loads the library, until the process exits.
static __device__ __align__(256) unsigned char
    g_static_scratch[STATIC_TABLE_BYTES + static_cast<size_t>(KT_STATIC_MAX_ELEMS) * sizeof(float)];

// Writes the tables into the scratch.  They travel as kernel parameters, which the runtime
// copies when the launch is queued: the call depends on no host memory after it returns.
__global__ void k_static_tables(const __grid_constant__ StaticTables tab, unsigned char *scratch) {
    const uint4 *src = reinterpret_cast<const uint4 *>(&tab);
    uint4 *dst = reinterpret_cast<uint4 *>(scratch);
    for (unsigned i = threadIdx.x; i < sizeof(StaticTables) / sizeof(uint4); i += blockDim.x) dst[i] = src[i];
}

constexpr int STATIC_MAX_DEVICES = 64;
std::mutex g_static_mutex;
unsigned char *g_static_addr[STATIC_MAX_DEVICES] = {};   // device address of the array, per device

}  // namespace

extern "C" int kt_sync_flat_static(const int32_t *group_of, const int32_t *shares, int K, int G,
                                   const void *const *grads, int in_dtype, int64_t n, void *out,
                                   int out_dtype, float scale, void *stream) {
    if (!group_of || !grads || !out) return fail(KT_ERR_INVALID, "NULL argument");
    if (K < 1 || K > KT_MAX_RANKS) return fail(KT_ERR_INVALID, "K = %d outside [1, %d]", K, KT_MAX_RANKS);
    if (G < 1 || G > KT_MAX_GROUPS || G > K) return fail(KT_ERR_INVALID, "G = %d outside [1, min(K, %d)]", G, KT_MAX_GROUPS);
    if (int rc = check_shares(shares, K)) return rc;
    if ((in_dtype != KT_F32 && in_dtype != KT_BF16) || (out_dtype != KT_F32 && out_dtype != KT_BF16))
        return fail(KT_ERR_INVALID, "unknown dtype");
    if (n < 1) return fail(KT_ERR_INVALID, "n = %lld must be >= 1", static_cast<long long>(n));
    const int64_t stride = round_up(n, 64);          // elements of one group's partial
    if (stride * G > KT_STATIC_MAX_ELEMS)
        return fail(KT_ERR_SHAPE,
                    "n = %lld with G = %d needs %lld fp32 scratch elements; the static scratch holds %d "
                    "(use kt_hier_reduce with caller-allocated transport buffers for larger problems)",
                    static_cast<long long>(n), G, static_cast<long long>(stride * G), KT_STATIC_MAX_ELEMS);
    const size_t es_in = in_dtype == KT_F32 ? 4 : 2, es_out = out_dtype == KT_F32 ? 4 : 2;
    if (reinterpret_cast<uintptr_t>(out) % es_out) return fail(KT_ERR_ALIGN, "out is not element aligned");

    // weights, in group-major rank order; everything on the stack
    int64_t Bg[KT_MAX_GROUPS] = {};
    int64_t B = 0;
    for (int r = 0; r < K; ++r) {
        if (group_of[r] < 0 || group_of[r] >= G) return fail(KT_ERR_INVALID, "group_of[%d] = %d outside [0, %d)", r, group_of[r], G);
        if (!grads[r]) return fail(KT_ERR_INVALID, "grads[%d] is NULL", r);
        if (reinterpret_cast<uintptr_t>(grads[r]) % es_in) return fail(KT_ERR_ALIGN, "grads[%d] is not element aligned", r);
        Bg[group_of[r]] += shares[r];
        B += shares[r];
    }
    for (int g = 0; g < G; ++g)
        if (!Bg[g]) return fail(KT_ERR_INVALID, "group %d has no rank", g);

    StaticTables tab;
    std::memset(&tab, 0, sizeof(tab));
    K1Params p1{};
    K2Params p2{};
    p1.rt.K = K;
    p2.gt.G = G;
    bool all_aligned = true;
    int k = 0;
    for (int g = 0; g < G; ++g) {
        bool first = true;
        for (int r = 0; r < K; ++r) {
            if (group_of[r] != g) continue;
            p1.rt.coef[k] = static_cast<float>(static_cast<double>(shares[r]) / static_cast<double>(Bg[g]));
            p1.rt.gid[k] = static_cast<signed char>(g);
            p1.rt.first[k] = first;
            p1.rt.last[k] = 0;
            tab.in_ptrs[k] = grads[r];
            all_aligned = all_aligned && aligned16(grads[r]);
            first = false;
            ++k;
        }
        p1.rt.last[k - 1] = 1;
        p2.gt.W[g] = static_cast<float>(static_cast<double>(Bg[g]) / static_cast<double>(B));
    }
    const int tile = in_dtype == KT_F32 ? TILE_F32 : TILE_BF16;
    const int n_tiles = static_cast<int>((stride + tile - 1) / tile);
    tab.prefix[0] = 0;
    tab.prefix[1] = n_tiles;
    tab.info.dst_off = 0;
    tab.info.numel = n;
    tab.info.ext = stride;
    tab.info.flags = all_aligned ? FLAG_ALIGNED : 0;
    tab.out_ptr[0] = out;
    tab.out_aligned[0] = aligned16(out) ? 1 : 0;

    // set-up, once per device: the array's name is only a host-side stand-in; kernels need
    // the device address the runtime reports for it on the current device
    int dev = 0;
    KT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return fail(KT_ERR_INVALID, "device ordinal %d not supported", dev);
    unsigned char *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_addr[dev]) {
            void *sym = nullptr;
            KT_CUDA(cudaGetSymbolAddress(&sym, g_static_scratch));
            g_static_addr[dev] = static_cast<unsigned char *>(sym);
        }
        scratch = g_static_addr[dev];
    }

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    k_static_tables<<<1, 64, 0, s>>>(tab, scratch);
    KT_CUDA(cudaGetLastError());

    TilePlan tp{};
    tp.prefix = reinterpret_cast<const int *>(scratch + offsetof(StaticTables, prefix));
    tp.info = reinterpret_cast<const TInfo *>(scratch + offsetof(StaticTables, info));
    tp.T = 1;
    tp.u_lo = 0;
    tp.u_hi = 1;
    tp.tile_lo = 0;
    tp.n_tiles = n_tiles;
    tp.tile = tile;
    tp.single = 1;
    tp.one = tab.info;
    float *partials = reinterpret_cast<float *>(scratch + STATIC_TABLE_BYTES);
    p1.tp = tp;
    p1.ptrs = reinterpret_cast<const void *const *>(scratch + offsetof(StaticTables, in_ptrs));
    p2.tp = tp;
    p2.out_ptrs = reinterpret_cast<void *const *>(scratch + offsetof(StaticTables, out_ptr));
    p2.out_aligned = scratch + offsetof(StaticTables, out_aligned);
    p2.R = 1;
    p2.scale = scale;
    p1.wide = p2.wide = 1;             // the partials start 4096 bytes into a 256-byte aligned array
    for (int g = 0; g < G; ++g) {
        p1.transport[g] = partials + g * stride;
        p2.src[g] = partials + g * stride;
    }
    // the reduce writes every element of the partials it uses, padding included, so nothing
    // left over from an earlier call is ever read
    if (in_dtype == KT_F32) k1_intra_reduce<float, float, KT_KB><<<n_tiles, NT, 0, s>>>(p1);
    else k1_intra_reduce<unsigned short, float, KT_KB><<<n_tiles, NT, 0, s>>>(p1);
    KT_CUDA(cudaGetLastError());
    if (out_dtype == KT_F32) launch_k2<float>(tile, n_tiles, s, p2);
    else launch_k2<unsigned short>(tile, n_tiles, s, p2);
    KT_CUDA(cudaGetLastError());
    return KT_OK;
}
