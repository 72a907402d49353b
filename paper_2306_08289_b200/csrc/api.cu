// C ABI of the engine: handle, plans, validation, descriptor upload, launches.
#include <cuda_runtime.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "a2cid2_internal.h"

namespace a2 {

namespace {
thread_local std::string g_thread_error = "";
}

void set_thread_error(const std::string& msg) { g_thread_error = msg; }
const char* thread_error() { return g_thread_error.c_str(); }

}  // namespace a2

using a2::DevItem;
using a2::DevOp;

namespace {

struct LaunchRange {
    int64_t item0, item1;  // items of the plan covered by this launch
    int64_t op0, op1;
    int workers = 2;  // most workers any item of the launch holds
    bool reloads = false;  // some operation fetches a gradient row in the middle of its item
};

// Grow-only pinned + device buffer pair used to ship the descriptors of one apply_events call.
struct Arena {
    void* host = nullptr;  // pinned
    void* dev = nullptr;
    size_t cap = 0;
    cudaEvent_t copied = nullptr;  // recorded after the last H2D copy out of `host`
    bool in_flight = false;
};

size_t elem_bytes(int32_t dtype) { return dtype == A2_BF16 ? 2 : 4; }

}  // namespace

struct a2cid2 {
    int32_t n = 0;
    int64_t d = 0;
    double eta = 0, alpha = 0, alpha_tilde = 0, gamma = 0;
    int32_t dtype = A2_F32;
    int32_t variant = A2_MSG_AFTER_MIX;
    int32_t item_workers = a2::kMaxItemWorkers;  // most workers A2_SCHED_CHAIN puts into one item (before the kernels' limits)
    int32_t launch_mode = A2_LAUNCH_AUTO;
    int32_t rounding = A2_ROUND_PER_EVENT;
    // borrowed buffers
    void* x = nullptr;
    void* xt = nullptr;
    void* g = nullptr;
    int32_t n_slots = 0;
    int64_t pitch = 0;
    cudaStream_t stream = nullptr;
    bool bound = false;
    int device = -1;
    // host-side times (authoritative; the kernels get them through the descriptors)
    std::vector<double> t;
    // library-owned scratch
    a2::DeviceInfo dev;
    bool dev_ok = false;
    double* d_partials = nullptr;  // consensus_grid doubles + 1 result
    double* d_dt = nullptr;        // n doubles
    double* h_pinned = nullptr;    // n + 1 doubles: dt staging and the result
    Arena arena[2];
    int arena_next = 0;
    std::vector<a2cid2_plan*> plans;  // live plans made from this handle
    uint64_t bind_epoch = 0;          // bumped whenever buffers, stream or variant change (invalidates plan graphs)
    cudaStream_t capture_stream = nullptr;  // private stream on which plan graphs are recorded
    std::string err;
};

// How a schedule is laid out in one descriptor blob, and how it is launched.
struct Packed {
    size_t bytes = 0;    // whole blob
    size_t ops_off = 0;  // DevOp array (the DevItem array sits at offset 0)
    // batched mode
    std::vector<LaunchRange> launches;
    std::vector<int64_t> batch_launch_first;  // launches of batch b: [first[b], first[b+1])
    std::vector<LaunchRange> slice_launches;  // the whole schedule as column-slice launches (items of several batches each)
    bool auto_slices = false;                 // what A2_LAUNCH_AUTO picks for a whole run of this schedule
    // resident mode
    bool resident = false;
    int32_t cache_rows = 0;
    size_t chunks_off = 0, g_rows_off = 0, events_off = 0;
    std::vector<a2::ResChunk> chunks;
    std::vector<int32_t> g_rows, cache_idx;
};

struct a2cid2_plan {
    a2cid2* owner = nullptr;
    a2cid2_sched* sched = nullptr;
    void* d_desc = nullptr;  // the descriptor blob on the device
    Packed pk;
    cudaGraphExec_t graph = nullptr;  // all launches of the plan as one CUDA graph (built on first whole run)
    uint64_t graph_epoch = 0;
    int64_t next_batch = 0;
    bool uses_gradients = false;
    std::vector<double> t_expect;  // workers' times the next batch expects
};

namespace {

int fail(a2cid2* h, int code, const std::string& msg) {
    if (h) h->err = msg;
    a2::set_thread_error(msg);
    return code;
}

int fail_cuda(a2cid2* h, cudaError_t e, const char* what) {
    std::string m = std::string(what) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")";
    return fail(h, A2_ECUDA, m);
}

#define A2_CUDA(h, call)                                         \
    do {                                                         \
        cudaError_t e__ = (call);                                \
        if (e__ != cudaSuccess) return fail_cuda(h, e__, #call); \
    } while (0)

int ensure_device(a2cid2* h) {
    if (h->dev_ok) return A2_OK;
    int rc = a2::query_device(&h->dev);
    if (rc != 0) return fail_cuda(h, (cudaError_t)rc, "device query");
    A2_CUDA(h, cudaGetDevice(&h->device));
    const int np = a2::consensus_grid(h->dev);
    A2_CUDA(h, cudaMalloc(&h->d_partials, sizeof(double) * (size_t)(np + 1)));
    A2_CUDA(h, cudaMalloc(&h->d_dt, sizeof(double) * (size_t)h->n));
    A2_CUDA(h, cudaMallocHost(&h->h_pinned, sizeof(double) * (size_t)(h->n + 1)));
    h->dev_ok = true;
    return A2_OK;
}

int need_bound(a2cid2* h) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (!h->bound) return fail(h, A2_ESTATE, "no buffers bound (call a2cid2_bind first)");
    return A2_OK;
}

// Split every batch into launches that respect the per-launch caps.
void make_launches(const a2cid2_sched& s, std::vector<LaunchRange>& launches, std::vector<int64_t>& batch_first) {
    const int64_t nb = (int64_t)s.batch_first.size() - 1;
    batch_first.assign((size_t)nb + 1, 0);
    for (int64_t b = 0; b < nb; ++b) {
        batch_first[(size_t)b] = (int64_t)launches.size();
        int64_t i = s.batch_first[(size_t)b];
        const int64_t iend = s.batch_first[(size_t)b + 1];
        while (i < iend) {
            LaunchRange L{i, i, s.items[(size_t)i].first_op, s.items[(size_t)i].first_op, 2};
            while (L.item1 < iend && (L.item1 - L.item0) < a2::kMaxItemsPerLaunch &&
                   (L.op1 - L.op0) + s.items[(size_t)L.item1].n_ops <= a2::kMaxOpsPerLaunch) {
                L.op1 += s.items[(size_t)L.item1].n_ops;
                const a2::SchedItem& si = s.items[(size_t)L.item1];
                L.workers = std::max(L.workers, si.d >= 0 ? 4 : (si.c >= 0 ? 3 : 2));
                L.item1 += 1;
            }
            for (int64_t o = L.op0; o < L.op1 && !L.reloads; ++o) L.reloads = s.ops[(size_t)o].reload >= 0;
            launches.push_back(L);
            i = L.item1;
        }
    }
    batch_first[(size_t)nb] = (int64_t)launches.size();
}

// The whole schedule cut into launches at the per-launch caps only: in a column-slice launch every CTA walks the
// items in schedule order over columns of its own, so batch boundaries need no launch boundary.
void make_slice_launches(const a2cid2_sched& s, std::vector<LaunchRange>& launches) {
    const int64_t n = (int64_t)s.items.size();
    int64_t i = 0;
    while (i < n) {
        LaunchRange L{i, i, s.items[(size_t)i].first_op, s.items[(size_t)i].first_op, 2};
        while (L.item1 < n && (L.item1 - L.item0) < a2::kMaxItemsPerLaunch &&
               (L.op1 - L.op0) + s.items[(size_t)L.item1].n_ops <= a2::kMaxOpsPerLaunch) {
            const a2::SchedItem& si = s.items[(size_t)L.item1];
            L.op1 += si.n_ops;
            L.workers = std::max(L.workers, si.d >= 0 ? 4 : (si.c >= 0 ? 3 : 2));
            L.item1 += 1;
        }
        for (int64_t o = L.op0; o < L.op1 && !L.reloads; ++o) L.reloads = s.ops[(size_t)o].reload >= 0;
        launches.push_back(L);
        i = L.item1;
    }
}

size_t align16(size_t v) { return (v + 15) & ~size_t(15); }

constexpr int64_t kAutoSliceBatchBytes = int64_t(1) << 30;  // 1 GiB per batch: about 160 microseconds of HBM traffic

// Decide how the schedule is launched and lay its descriptors out. Resident schedules need the
// population to fit shared memory.
int plan_layout(a2cid2* h, const a2cid2_sched& s, Packed& pk) {
    pk.resident = (s.flags & A2_SCHED_RESIDENT) != 0;
    pk.ops_off = align16(s.items.size() * sizeof(DevItem));
    size_t end = pk.ops_off + s.ops.size() * sizeof(DevOp);
    if (pk.resident && h->variant == A2_NO_MOMENTUM)
        return fail(h, A2_EINVAL, "A2_SCHED_RESIDENT is not available for the A2_NO_MOMENTUM variant");
    if (!pk.resident) {
        make_launches(s, pk.launches, pk.batch_launch_first);
        make_slice_launches(s, pk.slice_launches);
        // A2_LAUNCH_AUTO: column slices where a batch is short work for the whole GPU -- its launch would last
        // tens of microseconds, so launch gaps and the tail of every launch weigh (measured: 1.1x to 1.7x the
        // events per second on the 16- and 4-worker workloads) -- and one launch per batch where a batch moves
        // gigabytes (there the two modes are within a percent, and round-robin units keep all CTAs on the same
        // few rows, which the no-momentum kernels on bf16 rows reward with 7 %).
        const int64_t nb = (int64_t)s.batch_first.size() - 1;
        if (nb > 0) {
            a2cid2_stats st{};
            a2::schedule_stats(s, 0, nb, h->d, (int32_t)elem_bytes(h->dtype), h->variant != A2_NO_MOMENTUM, &st);
            pk.auto_slices = st.bytes_moved / nb < kAutoSliceBatchBytes;
        }
    } else {
        pk.cache_rows = a2::resident_cache_rows(h->n, h->n_slots);
        if (pk.cache_rows <= 0)
            return fail(h, A2_EINVAL, "A2_SCHED_RESIDENT: the population does not fit shared memory (need 2 n + 16 <= 216)");
        a2::build_resident_chunks(s, pk.cache_rows, pk.chunks, pk.g_rows, pk.cache_idx);
        pk.chunks_off = align16(end);
        pk.g_rows_off = align16(pk.chunks_off + pk.chunks.size() * sizeof(a2::ResChunk));
        pk.events_off = align16(pk.g_rows_off + pk.g_rows.size() * sizeof(int32_t));
        end = pk.events_off + s.items.size() * sizeof(a2::ResEv);  // this part is written on the device
    }
    pk.bytes = s.items.empty() ? 0 : end;
    return A2_OK;
}

// Bytes of the blob that have to be copied to the device (the resident event records at its end are
// produced there).
size_t upload_bytes(const a2cid2_sched& s, const Packed& pk) {
    if (s.items.empty()) return 0;
    return pk.resident ? pk.events_off : pk.bytes;
}

void write_descriptors(const a2cid2_sched& s, const Packed& pk, void* dst) {
    DevItem* di = static_cast<DevItem*>(dst);
    DevOp* dop = reinterpret_cast<DevOp*>(static_cast<char*>(dst) + pk.ops_off);
    if (!pk.resident) {
        for (const LaunchRange& L : pk.launches)
            for (int64_t k = L.item0; k < L.item1; ++k) {
                const a2::SchedItem& it = s.items[(size_t)k];
                di[k] = DevItem{it.a, it.b, it.c, it.d, it.slot_a, it.slot_b, it.slot_c, it.slot_d,
                                (int32_t)it.first_op, it.n_ops};  // counted from the plan's first operation
            }
    } else {
        for (size_t k = 0; k < s.items.size(); ++k) {  // one operation per item; slot_b carries the cache index
            const a2::SchedItem& it = s.items[k];
            di[k] = DevItem{it.a, it.b, -1, -1, it.slot_a, pk.cache_idx[k], -1, -1, (int32_t)k, 1};
        }
        if (!pk.chunks.empty())
            std::memcpy(static_cast<char*>(dst) + pk.chunks_off, pk.chunks.data(), pk.chunks.size() * sizeof(a2::ResChunk));
        if (!pk.g_rows.empty())
            std::memcpy(static_cast<char*>(dst) + pk.g_rows_off, pk.g_rows.data(), pk.g_rows.size() * sizeof(int32_t));
    }
    for (size_t o = 0; o < s.ops.size(); ++o) {
        const a2::SchedOp& op = s.ops[o];
        dop[o] = DevOp{op.kind, op.reload, op.t, op.t_prev_a, op.t_prev_b};
    }
}

// Most workers per item the kernels of the handle's storage type and variant take: four with fp32 rows and the
// momentum buffer, three with bf16 rows or without x~.
int32_t kernel_item_workers(const a2cid2* h) { return (h->dtype == A2_F32 && h->variant != A2_NO_MOMENTUM) ? 4 : 3; }
int32_t item_workers(const a2cid2* h) {
    const int32_t cap = kernel_item_workers(h);
    return h->item_workers < cap ? h->item_workers : cap;
}

// Scheduling flags as the engine uses them: an item may change a worker's gradient row between two of its
// gradient operations exactly where the event kernels fetch rows operation by operation (fp32 rows).
uint32_t engine_flags(const a2cid2* h, uint32_t flags) {
    if (h->dtype == A2_F32) return flags | A2_SCHED_ROW_PER_OP;
    return flags & ~uint32_t(A2_SCHED_ROW_PER_OP);
}

// Column-slice launches serve a schedule that is run whole (any batch boundary inside a launch is then harmless);
// a range of batches is run with one launch per batch.
bool uses_slices(const a2cid2* h, const a2cid2_sched& s, const Packed& pk, int64_t b0, int64_t b1) {
    const int64_t nb = (int64_t)s.batch_first.size() - 1;
    if ((s.flags & A2_SCHED_RESIDENT) || b0 != 0 || b1 != nb) return false;
    if (h->launch_mode == A2_LAUNCH_AUTO) return pk.auto_slices;
    return h->launch_mode == A2_LAUNCH_COLUMN_SLICES;
}

// Queue the kernels of batches [b0, b1) of a schedule whose blob sits at `dev`.
int queue_batches(a2cid2* h, const a2cid2_sched& s, const Packed& pk, void* dev, int64_t b0, int64_t b1,
                  cudaStream_t stream) {
    if (b1 <= b0) return A2_OK;
    char* base = static_cast<char*>(dev);
    const DevItem* d_items = reinterpret_cast<const DevItem*>(base);
    const DevOp* d_ops = reinterpret_cast<const DevOp*>(base + pk.ops_off);
    if (pk.resident) {
        if (h->variant == A2_NO_MOMENTUM)
            return fail(h, A2_EINVAL, "A2_SCHED_RESIDENT is not available for the A2_NO_MOMENTUM variant");
        if (h->rounding == A2_ROUND_PER_STORE)
            return fail(h, A2_EINVAL, "A2_SCHED_RESIDENT rounds every value at every event: not available with A2_ROUND_PER_STORE");
        a2::ResidentLaunch L;
        L.x = h->x; L.xt = h->xt; L.g = h->g; L.pitch = h->pitch; L.d = h->d;
        L.n = h->n; L.dtype = h->dtype; L.variant = h->variant; L.eta = h->eta;
        L.alpha = (float)h->alpha; L.alpha_tilde = (float)h->alpha_tilde; L.gamma = (float)h->gamma;
        L.items = d_items; L.ops = d_ops;
        L.events = reinterpret_cast<a2::ResEv*>(base + pk.events_off);
        L.chunks = reinterpret_cast<const a2::ResChunk*>(base + pk.chunks_off);
        L.g_rows = reinterpret_cast<const int32_t*>(base + pk.g_rows_off);
        L.n_events = (int32_t)s.items.size(); L.n_chunks = (int32_t)pk.chunks.size(); L.cache_rows = pk.cache_rows;
        const int rc = a2::launch_resident(L, h->dev, stream);
        if (rc != 0) return fail_cuda(h, (cudaError_t)rc, "resident kernel launch");
        return A2_OK;
    }
    const bool per_store = h->rounding == A2_ROUND_PER_STORE;
    if (per_store) {  // before anything is launched
        if (h->variant == A2_NO_MOMENTUM) return fail(h, A2_ESTATE, "A2_ROUND_PER_STORE has no meaning for the A2_NO_MOMENTUM variant");
        if (!a2::rows_allow_256bit(h->x, h->xt, h->g, h->pitch, h->dtype))
            return fail(h, A2_ESTATE, "A2_ROUND_PER_STORE needs x, x_tilde and the gradient buffer on 32-byte boundaries and a row pitch that is a multiple of 32 bytes");
    }
    const std::vector<LaunchRange>& list = uses_slices(h, s, pk, b0, b1) ? pk.slice_launches : pk.launches;
    const bool slices = &list == &pk.slice_launches;
    const int64_t l0 = slices ? 0 : pk.batch_launch_first[(size_t)b0];
    const int64_t l1 = slices ? (int64_t)list.size() : pk.batch_launch_first[(size_t)b1];
    for (int64_t l = l0; l < l1; ++l)  // before anything is launched
        if (list[(size_t)l].workers > kernel_item_workers(h))
            return fail(h, A2_ESTATE, "this plan holds four-worker items, which the kernels of the current variant do not take");
    for (int64_t l = l0; l < l1; ++l) {
        const LaunchRange& R = list[(size_t)l];
        a2::EventLaunch L;
        L.x = h->x; L.xt = h->xt; L.g = h->g; L.pitch = h->pitch; L.d = h->d;
        L.items = d_items + R.item0;
        L.ops = d_ops + R.op0;
        L.n_items = (int32_t)(R.item1 - R.item0);
        L.n_ops = (int32_t)(R.op1 - R.op0);
        L.eta = h->eta;
        L.alpha = (float)h->alpha; L.alpha_tilde = (float)h->alpha_tilde; L.gamma = (float)h->gamma;
        L.variant = h->variant; L.dtype = h->dtype;
        L.max_workers = R.workers;
        L.op_base = (int32_t)R.op0;
        L.slice = slices;
        L.has_reloads = R.reloads;
        L.round_per_store = per_store;
        const int rc = a2::launch_events(L, h->dev, stream);
        if (rc != 0) return fail_cuda(h, (cudaError_t)rc, "event kernel launch");
    }
    return A2_OK;
}

constexpr int64_t kGraphMinLaunches = 4;

// Record all launches of a (batched) plan into a CUDA graph if that has not been done for the current
// binding, then launch the graph on the handle's stream.
int ensure_plan_graph(a2cid2* h, a2cid2_plan* p) {
    if (p->graph && p->graph_epoch != h->bind_epoch) {
        cudaGraphExecDestroy(p->graph);
        p->graph = nullptr;
    }
    if (!p->graph) {
        if (!h->capture_stream) A2_CUDA(h, cudaStreamCreateWithFlags(&h->capture_stream, cudaStreamNonBlocking));
        const int64_t nb = (int64_t)p->sched->batch_first.size() - 1;
        A2_CUDA(h, cudaStreamBeginCapture(h->capture_stream, cudaStreamCaptureModeThreadLocal));
        const int rc = queue_batches(h, *p->sched, p->pk, p->d_desc, 0, nb, h->capture_stream);
        cudaGraph_t g = nullptr;
        const cudaError_t e = cudaStreamEndCapture(h->capture_stream, &g);
        if (rc != A2_OK) { if (g) cudaGraphDestroy(g); return rc; }
        if (e != cudaSuccess) return fail_cuda(h, e, "cudaStreamEndCapture");
        const cudaError_t ei = cudaGraphInstantiate(&p->graph, g, 0);
        cudaGraphDestroy(g);
        if (ei != cudaSuccess) { p->graph = nullptr; return fail_cuda(h, ei, "cudaGraphInstantiate"); }
        p->graph_epoch = h->bind_epoch;
    }
    return A2_OK;
}

// Launches a whole run of the plan takes under the handle's launch mode.
int64_t whole_run_launches(const a2cid2* h, const a2cid2_plan* p) {
    const int64_t nb = (int64_t)p->sched->batch_first.size() - 1;
    return uses_slices(h, *p->sched, p->pk, 0, nb) ? (int64_t)p->pk.slice_launches.size() : (int64_t)p->pk.launches.size();
}

int run_plan_graph(a2cid2* h, a2cid2_plan* p) {
    const int rc = ensure_plan_graph(h, p);
    if (rc != A2_OK) return rc;
    A2_CUDA(h, cudaGraphLaunch(p->graph, h->stream));
    return A2_OK;
}

// Descriptor-derived counters of batches [b0, b1).
void fill_stats(const a2cid2* h, const a2cid2_sched& s, const Packed& pk, int64_t b0, int64_t b1, a2cid2_stats* st) {
    const int32_t eb = (int32_t)elem_bytes(h->dtype);
    a2::schedule_stats(s, b0, b1, h->d, eb, h->variant != A2_NO_MOMENTUM, st);
    if (pk.resident) {  // the state crosses HBM once each way, every cached gradient row once per chunk
        st->n_launches = b1 > b0 ? 2 : 0;
        st->bytes_moved = b1 > b0 ? ((int64_t)4 * h->n + (int64_t)pk.g_rows.size()) * h->d * eb : 0;
    } else {
        st->n_launches = uses_slices(h, s, pk, b0, b1) ? (int64_t)pk.slice_launches.size()
                                                   : pk.batch_launch_first[(size_t)b1] - pk.batch_launch_first[(size_t)b0];
    }
}

// After batches [b0, b1) ran: every worker's time is that of its last operation in them.
void advance_times(const a2cid2_sched& s, int64_t b0, int64_t b1, std::vector<double>& t) {
    for (int64_t k = s.batch_first[(size_t)b0]; k < s.batch_first[(size_t)b1]; ++k) {
        const a2::SchedItem& it = s.items[(size_t)k];
        for (int32_t o = 0; o < it.n_ops; ++o) {
            const a2::SchedOp& op = s.ops[(size_t)(it.first_op + o)];
            const int32_t k = op.kind;
            if (k == A2_OP_GRAD_A || k == A2_OP_MIX_A || k == A2_OP_COMM || k == A2_OP_COMM_AC || k == A2_OP_COMM_AD) t[(size_t)it.a] = op.t;
            if (k == A2_OP_GRAD_B || k == A2_OP_COMM || k == A2_OP_COMM_BC || k == A2_OP_COMM_BD) t[(size_t)it.b] = op.t;
            if (k == A2_OP_GRAD_C || k == A2_OP_COMM_AC || k == A2_OP_COMM_BC || k == A2_OP_COMM_CD) t[(size_t)it.c] = op.t;
            if (k == A2_OP_GRAD_D || k == A2_OP_COMM_AD || k == A2_OP_COMM_BD || k == A2_OP_COMM_CD) t[(size_t)it.d] = op.t;
        }
    }
}

bool needs_gradients(const a2cid2_sched& s) {
    for (const a2::SchedItem& it : s.items)
        if (it.slot_a >= 0 || it.slot_b >= 0 || it.slot_c >= 0 || it.slot_d >= 0) return true;
    return false;
}

double now_ms() {
    using namespace std::chrono;
    return duration<double, std::milli>(steady_clock::now().time_since_epoch()).count();
}

}  // namespace

extern "C" {

const char* a2cid2_version(void) { return "a2cid2-b200 0.1 (sm_100a)"; }

const char* a2cid2_last_error(const a2cid2_t* h) { return h ? h->err.c_str() : a2::thread_error(); }

int a2cid2_create(int32_t n, int64_t d, double eta, double alpha, double alpha_tilde, double gamma,
                  int32_t storage_dtype, a2cid2_t** out) {
    if (!out) return fail(nullptr, A2_EINVAL, "out is NULL");
    *out = nullptr;
    if (n < 2 || n > 4096) return fail(nullptr, A2_EINVAL, "need 2 <= n <= 4096 workers");
    if (d < 1 || d > (int64_t(1) << 40)) return fail(nullptr, A2_EINVAL, "need 1 <= d <= 2^40");
    if (!std::isfinite(eta) || !std::isfinite(alpha) || !std::isfinite(alpha_tilde) || !std::isfinite(gamma))
        return fail(nullptr, A2_EINVAL, "hyper-parameters must be finite");
    if (eta < 0) return fail(nullptr, A2_EINVAL, "eta must be >= 0");
    if (storage_dtype != A2_F32 && storage_dtype != A2_BF16) return fail(nullptr, A2_EINVAL, "unknown storage type");
    a2cid2* h = new (std::nothrow) a2cid2();
    if (!h) return fail(nullptr, A2_ENOMEM, "out of host memory");
    h->n = n; h->d = d; h->eta = eta; h->alpha = alpha; h->alpha_tilde = alpha_tilde; h->gamma = gamma;
    h->dtype = storage_dtype;
    if (const char* v = a2::tuning_env("A2CID2_ITEM_WORKERS")) {  // tuning override
        const int k = std::atoi(v);
        if (k >= 2 && k <= a2::kMaxItemWorkers) h->item_workers = k;
    }
    h->t.assign((size_t)n, 0.0);
    *out = h;
    return A2_OK;
}

int a2cid2_set_variant(a2cid2_t* h, int32_t variant) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (variant != A2_MSG_AFTER_MIX && variant != A2_MSG_BEFORE_MIX && variant != A2_NO_MOMENTUM)
        return fail(h, A2_EINVAL, "unknown variant");
    if (variant != A2_NO_MOMENTUM && h->bound && !h->xt)
        return fail(h, A2_ESTATE, "this variant needs an x_tilde buffer and none is bound");
    h->variant = variant;
    h->bind_epoch += 1;
    return A2_OK;
}

int a2cid2_set_launch_mode(a2cid2_t* h, int32_t mode) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (mode != A2_LAUNCH_AUTO && mode != A2_LAUNCH_PER_BATCH && mode != A2_LAUNCH_COLUMN_SLICES)
        return fail(h, A2_EINVAL, "unknown launch mode");
    h->launch_mode = mode;
    h->bind_epoch += 1;  // recorded plan graphs hold the launches of the previous mode
    return A2_OK;
}

int a2cid2_set_rounding(a2cid2_t* h, int32_t mode) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (mode != A2_ROUND_PER_EVENT && mode != A2_ROUND_PER_STORE) return fail(h, A2_EINVAL, "unknown rounding mode");
    if (mode == A2_ROUND_PER_STORE && h->dtype != A2_F32)
        return fail(h, A2_EINVAL, "A2_ROUND_PER_STORE is for fp32 rows (bf16 rows are rounded to eight bits at every store anyway)");
    h->rounding = mode;
    h->bind_epoch += 1;  // recorded plan graphs hold the kernels of the previous mode
    return A2_OK;
}

int a2cid2_bind(a2cid2_t* h, void* x, void* x_tilde, void* grads, int32_t n_grad_slots, int64_t row_pitch_elems,
                void* cuda_stream) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (!x) return fail(h, A2_EINVAL, "x is NULL");
    if (!x_tilde && h->variant != A2_NO_MOMENTUM)
        return fail(h, A2_EINVAL, "x_tilde is NULL (only the A2_NO_MOMENTUM variant runs without it)");
    if (n_grad_slots < 0 || (n_grad_slots > 0 && !grads)) return fail(h, A2_EINVAL, "bad gradient buffer");
    if (row_pitch_elems < h->d || row_pitch_elems % 8 != 0)
        return fail(h, A2_EINVAL, "row pitch must be >= d and a multiple of 8 elements");
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(x_tilde) | reinterpret_cast<uintptr_t>(grads)) & 15)
        return fail(h, A2_EINVAL, "buffers must be 16-byte aligned");
    if (x == x_tilde) return fail(h, A2_EINVAL, "x and x_tilde must be distinct buffers");
    const int rc = ensure_device(h);
    if (rc != A2_OK) return rc;
    h->x = x; h->xt = x_tilde; h->g = n_grad_slots > 0 ? grads : nullptr;
    h->n_slots = n_grad_slots; h->pitch = row_pitch_elems;
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    h->bound = true;
    h->bind_epoch += 1;
    return A2_OK;
}

int a2cid2_write_state(a2cid2_t* h, const void* host_x, const void* host_x_tilde, const double* host_t) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!host_x) return fail(h, A2_EINVAL, "host_x is NULL");
    if (host_x_tilde && !h->xt) return fail(h, A2_EINVAL, "host_x_tilde given but no x_tilde buffer is bound");
    if (host_t)
        for (int32_t w = 0; w < h->n; ++w)
            if (!std::isfinite(host_t[w])) return fail(h, A2_EINVAL, "non-finite worker time");
    const size_t eb = elem_bytes(h->dtype);
    const size_t row = (size_t)h->d * eb, pitch = (size_t)h->pitch * eb;
    A2_CUDA(h, cudaMemcpy2DAsync(h->x, pitch, host_x, row, row, (size_t)h->n, cudaMemcpyHostToDevice, h->stream));
    if (h->xt)
        A2_CUDA(h, cudaMemcpy2DAsync(h->xt, pitch, host_x_tilde ? host_x_tilde : host_x, row, row, (size_t)h->n,
                                     cudaMemcpyHostToDevice, h->stream));
    A2_CUDA(h, cudaStreamSynchronize(h->stream));
    for (int32_t w = 0; w < h->n; ++w) h->t[(size_t)w] = host_t ? host_t[w] : 0.0;
    return A2_OK;
}

int a2cid2_write_grads(a2cid2_t* h, int32_t first_slot, int32_t n_slots, const void* host_g) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!host_g || first_slot < 0 || n_slots < 0 || first_slot + n_slots > h->n_slots)
        return fail(h, A2_ERANGE, "gradient slot range out of bounds");
    if (n_slots == 0) return A2_OK;
    const size_t eb = elem_bytes(h->dtype);
    const size_t row = (size_t)h->d * eb, pitch = (size_t)h->pitch * eb;
    char* dst = static_cast<char*>(h->g) + (size_t)first_slot * pitch;
    A2_CUDA(h, cudaMemcpy2DAsync(dst, pitch, host_g, row, row, (size_t)n_slots, cudaMemcpyHostToDevice, h->stream));
    A2_CUDA(h, cudaStreamSynchronize(h->stream));
    return A2_OK;
}

int a2cid2_read_state(a2cid2_t* h, void* host_x, void* host_x_tilde, double* host_t) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (host_x_tilde && !h->xt) return fail(h, A2_ESTATE, "no x_tilde buffer is bound");
    const size_t eb = elem_bytes(h->dtype);
    const size_t row = (size_t)h->d * eb, pitch = (size_t)h->pitch * eb;
    if (host_x)
        A2_CUDA(h, cudaMemcpy2DAsync(host_x, row, h->x, pitch, row, (size_t)h->n, cudaMemcpyDeviceToHost, h->stream));
    if (host_x_tilde)
        A2_CUDA(h, cudaMemcpy2DAsync(host_x_tilde, row, h->xt, pitch, row, (size_t)h->n, cudaMemcpyDeviceToHost, h->stream));
    A2_CUDA(h, cudaStreamSynchronize(h->stream));
    if (host_t) std::memcpy(host_t, h->t.data(), sizeof(double) * (size_t)h->n);
    return A2_OK;
}

int a2cid2_times(const a2cid2_t* h, double* host_t) {
    if (!h || !host_t) return fail(nullptr, A2_EINVAL, "NULL argument");
    std::memcpy(host_t, h->t.data(), sizeof(double) * (size_t)h->n);
    return A2_OK;
}

int a2cid2_set_times(a2cid2_t* h, const double* host_t) {
    if (!h || !host_t) return fail(h, A2_EINVAL, "NULL argument");
    for (int32_t w = 0; w < h->n; ++w)
        if (!std::isfinite(host_t[w])) return fail(h, A2_EINVAL, "non-finite worker time");
    for (int32_t w = 0; w < h->n; ++w) h->t[(size_t)w] = host_t[w];
    return A2_OK;
}

// Lay out, upload and queue a whole schedule through the handle's staging buffers; takes ownership of s.
static int submit_schedule(a2cid2* h, a2cid2_sched* s, a2cid2_stats* stats, double t0) {
    Packed pk;
    int rc = plan_layout(h, *s, pk);
    if (rc != A2_OK) { a2cid2_sched_destroy(s); return rc; }
    const int64_t nb = (int64_t)s->batch_first.size() - 1;
    if (stats) std::memset(stats, 0, sizeof *stats);
    if (pk.bytes > 0) {
        Arena& A = h->arena[h->arena_next];
        h->arena_next ^= 1;
        if (A.in_flight) {  // the previous copy out of this staging buffer must have finished
            cudaError_t e = cudaEventSynchronize(A.copied);
            if (e != cudaSuccess) { a2cid2_sched_destroy(s); return fail_cuda(h, e, "cudaEventSynchronize"); }
            A.in_flight = false;
        }
        if (A.cap < pk.bytes) {
            // the device side may still be read by queued kernels: wait before freeing it
            cudaError_t e = cudaStreamSynchronize(h->stream);
            if (e == cudaSuccess && A.host) e = cudaFreeHost(A.host);
            if (e == cudaSuccess && A.dev) e = cudaFree(A.dev);
            A.host = A.dev = nullptr;
            A.cap = 0;
            const size_t cap = pk.bytes + pk.bytes / 2 + 4096;
            if (e == cudaSuccess) e = cudaMallocHost(&A.host, cap);
            if (e == cudaSuccess) e = cudaMalloc(&A.dev, cap);
            if (e == cudaSuccess && !A.copied) e = cudaEventCreateWithFlags(&A.copied, cudaEventDisableTiming);
            if (e != cudaSuccess) { a2cid2_sched_destroy(s); return fail_cuda(h, e, "descriptor buffer allocation"); }
            A.cap = cap;
        }
        write_descriptors(*s, pk, A.host);
        const size_t up = upload_bytes(*s, pk);
        cudaError_t e = cudaMemcpyAsync(A.dev, A.host, up, cudaMemcpyHostToDevice, h->stream);
        if (e == cudaSuccess) e = cudaEventRecord(A.copied, h->stream);
        if (e != cudaSuccess) { a2cid2_sched_destroy(s); return fail_cuda(h, e, "descriptor upload"); }
        A.in_flight = true;
        const double t1 = now_ms();
        rc = queue_batches(h, *s, pk, A.dev, 0, nb, h->stream);
        if (rc != A2_OK) { a2cid2_sched_destroy(s); return rc; }
        if (stats) {
            fill_stats(h, *s, pk, 0, nb, stats);
            stats->descriptor_bytes = (int64_t)up;
            stats->host_ms = t1 - t0;
        }
    }
    h->t = s->t_final;
    a2cid2_sched_destroy(s);
    return A2_OK;
}

int a2cid2_apply_events(a2cid2_t* h, int64_t n_events, const double* times, const int32_t* wi, const int32_t* wj,
                        const int32_t* grad_slot, uint32_t flags, a2cid2_stats* stats) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    const double t0 = now_ms();
    a2cid2_sched* s = nullptr;
    std::string err;
    rc = a2::build_schedule(h->n, h->n_slots, h->t.data(), n_events, times, wi, wj, grad_slot, engine_flags(h, flags), 0, item_workers(h),
                            &s, err);
    if (rc != A2_OK) return fail(h, rc, err);
    return submit_schedule(h, s, stats, t0);
}

int a2cid2_flush(a2cid2_t* h, double t_flush) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!std::isfinite(t_flush)) return fail(h, A2_EINVAL, "t_flush must be finite");
    for (int32_t w = 0; w < h->n; ++w)
        if (t_flush < h->t[(size_t)w]) return fail(h, A2_EORDER, "t_flush precedes a worker's last event");
    if (h->variant == A2_NO_MOMENTUM) {  // no flow between events: only the clock moves
        h->t.assign((size_t)h->n, t_flush);
        return A2_OK;
    }
    a2cid2_sched* s = new (std::nothrow) a2cid2_sched();
    if (!s) return fail(h, A2_ENOMEM, "out of host memory");
    s->n = h->n;
    s->n_grad_slots = h->n_slots;
    s->t_start = h->t;
    s->t_final = h->t;
    for (int32_t w = 0; w < h->n; ++w) {  // one batch: a mixing-only item per worker that is behind
        if (h->t[(size_t)w] == t_flush) continue;
        s->items.push_back(a2::SchedItem{w, -1, -1, -1, -1, -1, -1, -1, (int64_t)s->ops.size(), 1, 0});
        s->ops.push_back(a2::SchedOp{-1, A2_OP_MIX_A, t_flush, h->t[(size_t)w], 0.0});
        s->t_final[(size_t)w] = t_flush;
    }
    s->batch_first.assign(1, 0);
    if (!s->items.empty()) s->batch_first.push_back((int64_t)s->items.size());
    return submit_schedule(h, s, nullptr, now_ms());
}

int a2cid2_consensus_distance(a2cid2_t* h, double t_eval, double* out) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!out) return fail(h, A2_EINVAL, "out is NULL");
    bool flush = !std::isnan(t_eval);
    const int np = a2::consensus_grid(h->dev);
    if (flush) {
        if (!std::isfinite(t_eval)) return fail(h, A2_EINVAL, "t_eval must be finite or NaN");
        for (int32_t w = 0; w < h->n; ++w)
            if (t_eval < h->t[(size_t)w]) return fail(h, A2_EORDER, "t_eval precedes a worker's last event");
        if (h->variant == A2_NO_MOMENTUM) flush = false;  // the rows do not move between events
    }
    if (flush) {
        // the staging buffer is free: every earlier call waited for the stream before returning
        for (int32_t w = 0; w < h->n; ++w) h->h_pinned[w] = t_eval - h->t[(size_t)w];
        A2_CUDA(h, cudaMemcpyAsync(h->d_dt, h->h_pinned, sizeof(double) * (size_t)h->n, cudaMemcpyHostToDevice, h->stream));
    }
    const int lrc = a2::launch_consensus(h->x, h->xt, h->pitch, h->n, h->d, h->dtype, h->eta, flush ? h->d_dt : nullptr,
                                         h->d_partials, np, h->d_partials + np, h->stream);
    if (lrc != 0) return fail_cuda(h, (cudaError_t)lrc, "consensus kernel launch");
    A2_CUDA(h, cudaMemcpyAsync(h->h_pinned + h->n, h->d_partials + np, sizeof(double), cudaMemcpyDeviceToHost, h->stream));
    A2_CUDA(h, cudaStreamSynchronize(h->stream));
    *out = h->h_pinned[h->n];
    return A2_OK;
}

int a2cid2_sync(a2cid2_t* h) {
    if (!h) return fail(nullptr, A2_EINVAL, "handle is NULL");
    if (!h->dev_ok) return A2_OK;
    A2_CUDA(h, cudaStreamSynchronize(h->stream));
    return A2_OK;
}

void a2cid2_destroy(a2cid2_t* h) {
    if (!h) return;
    if (h->dev_ok) cudaStreamSynchronize(h->stream);
    // plans that outlive the handle keep their memory until a2cid2_plan_destroy, but can no longer run
    for (a2cid2_plan* p : h->plans) p->owner = nullptr;
    if (h->dev_ok) {
        for (Arena& A : h->arena) {
            if (A.host) cudaFreeHost(A.host);
            if (A.dev) cudaFree(A.dev);
            if (A.copied) cudaEventDestroy(A.copied);
        }
        if (h->capture_stream) cudaStreamDestroy(h->capture_stream);
        if (h->d_partials) cudaFree(h->d_partials);
        if (h->d_dt) cudaFree(h->d_dt);
        if (h->h_pinned) cudaFreeHost(h->h_pinned);
    }
    delete h;
}

int a2cid2_consensus_distance_static(const void* x, int32_t n, int64_t d, int64_t row_pitch_elems, int32_t storage_dtype,
                                     void* cuda_stream, double* out_device) {
    if (!x || !out_device) return fail(nullptr, A2_EINVAL, "x or out_device is NULL");
    if (storage_dtype != A2_F32 && storage_dtype != A2_BF16) return fail(nullptr, A2_EINVAL, "unknown storage type");
    if (n < 2 || n > 4096) return fail(nullptr, A2_EINVAL, "need 2 <= n <= 4096 workers");
    if (d < 1) return fail(nullptr, A2_EINVAL, "need d >= 1");
    if (row_pitch_elems < d || row_pitch_elems % 8 != 0)
        return fail(nullptr, A2_EINVAL, "row pitch must be >= d and a multiple of 8 elements");
    if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(out_device) & 7))
        return fail(nullptr, A2_EINVAL, "x must be 16-byte aligned and out_device 8-byte aligned");
    const int64_t max_d = a2::consensus_static_max_columns(storage_dtype);
    if (d > max_d) {
        char buf[200];
        std::snprintf(buf, sizeof buf,
                      "d = %lld exceeds the %lld columns the fixed scratch array of this entry point covers; "
                      "use a2cid2_consensus_distance",
                      (long long)d, (long long)max_d);
        return fail(nullptr, A2_ERANGE, buf);
    }
    const int rc = a2::launch_consensus_static(x, row_pitch_elems, n, d, storage_dtype, out_device, cuda_stream, nullptr);
    if (rc != 0) return fail_cuda(nullptr, (cudaError_t)rc, "static consensus launch");
    return A2_OK;
}

// ---- plans -----------------------------------------------------------------------------------

int a2cid2_plan_create(a2cid2_t* h, const double* t_start, int64_t n_events, const double* times, const int32_t* wi,
                       const int32_t* wj, const int32_t* grad_slot, uint32_t flags, a2cid2_plan_t** out) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!out) return fail(h, A2_EINVAL, "out is NULL");
    *out = nullptr;
    a2cid2_sched* s = nullptr;
    std::string err;
    rc = a2::build_schedule(h->n, h->n_slots, t_start ? t_start : h->t.data(), n_events, times, wi, wj, grad_slot,
                            engine_flags(h, flags), 0, item_workers(h), &s, err);
    if (rc != A2_OK) return fail(h, rc, err);
    a2cid2_plan* p = new (std::nothrow) a2cid2_plan();
    if (!p) { a2cid2_sched_destroy(s); return fail(h, A2_ENOMEM, "out of host memory"); }
    p->owner = h;
    p->sched = s;
    p->t_expect = s->t_start;
    p->uses_gradients = needs_gradients(*s);
    rc = plan_layout(h, *s, p->pk);
    if (rc != A2_OK) { a2cid2_sched_destroy(s); delete p; return rc; }
    if (p->pk.bytes > 0) {
        const size_t up = upload_bytes(*s, p->pk);
        std::vector<char> staging(up);
        write_descriptors(*s, p->pk, staging.data());
        cudaError_t e = cudaMalloc(&p->d_desc, p->pk.bytes);
        // pageable source: the copy has left the host buffer when the call returns
        if (e == cudaSuccess) e = cudaMemcpy(p->d_desc, staging.data(), up, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            if (p->d_desc) cudaFree(p->d_desc);
            a2cid2_sched_destroy(s);
            delete p;
            return fail_cuda(h, e, "plan descriptor upload");
        }
    }
    if (!p->pk.resident && whole_run_launches(h, p) >= kGraphMinLaunches) {
        rc = ensure_plan_graph(h, p);  // recorded now, so that running the plan is a single submission
        if (rc != A2_OK) {
            if (p->d_desc) cudaFree(p->d_desc);
            a2cid2_sched_destroy(s);
            delete p;
            return rc;
        }
    }
    h->plans.push_back(p);
    *out = p;
    return A2_OK;
}

const a2cid2_sched_t* a2cid2_plan_sched(const a2cid2_plan_t* p) { return p ? p->sched : nullptr; }

int a2cid2_plan_run(a2cid2_t* h, a2cid2_plan_t* p, int64_t first_batch, int64_t n_batches, a2cid2_stats* stats) {
    int rc = need_bound(h);
    if (rc != A2_OK) return rc;
    if (!p || p->owner != h) return fail(h, A2_EINVAL, "plan is NULL or belongs to another handle");
    const int64_t nb = (int64_t)p->sched->batch_first.size() - 1;
    if (n_batches < 0) n_batches = nb - first_batch;
    if (first_batch != p->next_batch) return fail(h, A2_ESTATE, "plan batches must be run in order, each once");
    if (first_batch < 0 || n_batches < 0 || first_batch + n_batches > nb) return fail(h, A2_ERANGE, "batch range out of bounds");
    if (p->t_expect != h->t) return fail(h, A2_ESTATE, "the handle's worker times are not those the plan starts from");
    if (p->uses_gradients && !h->g) return fail(h, A2_ESTATE, "plan has gradient events but no gradient buffer is bound");
    const int64_t b1 = first_batch + n_batches;
    if (n_batches > 0) {
        // A plan of several launches run whole goes out as one CUDA graph: one submission instead of one per
        // batch. The graph was recorded on a private stream when the plan was made and is recorded again only if
        // the bound buffers, the stream or the variant have changed since.
        const bool whole = first_batch == 0 && b1 == nb;
        if (whole && !p->pk.resident && whole_run_launches(h, p) >= kGraphMinLaunches) {
            rc = run_plan_graph(h, p);
        } else {
            rc = queue_batches(h, *p->sched, p->pk, p->d_desc, first_batch, b1, h->stream);
        }
        if (rc != A2_OK) return rc;
        advance_times(*p->sched, first_batch, b1, h->t);
    }
    p->next_batch = b1;
    p->t_expect = h->t;
    if (stats) {
        fill_stats(h, *p->sched, p->pk, first_batch, b1, stats);
        stats->descriptor_bytes = 0;
        stats->host_ms = 0.0;
    }
    return A2_OK;
}

void a2cid2_plan_destroy(a2cid2_plan_t* p) {
    if (!p) return;
    if (p->owner) {
        if (p->owner->dev_ok) cudaStreamSynchronize(p->owner->stream);  // queued kernels may still read the descriptors
        std::vector<a2cid2_plan*>& v = p->owner->plans;
        for (size_t k = 0; k < v.size(); ++k)
            if (v[k] == p) { v.erase(v.begin() + (long)k); break; }
    }
    if (p->graph) cudaGraphExecDestroy(p->graph);
    if (p->d_desc) cudaFree(p->d_desc);
    a2cid2_sched_destroy(p->sched);
    delete p;
}

// ---- host scheduler ----------------------------------------------------------------------------

int a2cid2_sched_create(int32_t n, int32_t n_grad_slots, const double* t_last, int64_t n_events, const double* times,
                        const int32_t* wi, const int32_t* wj, const int32_t* grad_slot, uint32_t flags,
                        int32_t max_ops_per_item, int32_t max_workers_per_item, a2cid2_sched_t** out) {
    std::string err;
    const int rc = a2::build_schedule(n, n_grad_slots, t_last, n_events, times, wi, wj, grad_slot, flags, max_ops_per_item,
                                      max_workers_per_item, out, err);
    if (rc != A2_OK) a2::set_thread_error(err);
    return rc;
}

int64_t a2cid2_sched_num_batches(const a2cid2_sched_t* s) { return s ? (int64_t)s->batch_first.size() - 1 : 0; }
int64_t a2cid2_sched_num_items(const a2cid2_sched_t* s) { return s ? (int64_t)s->items.size() : 0; }
int64_t a2cid2_sched_num_ops(const a2cid2_sched_t* s) { return s ? (int64_t)s->ops.size() : 0; }

int a2cid2_sched_batch_items(const a2cid2_sched_t* s, int64_t b, int64_t* first_item, int64_t* n_items) {
    if (!s || !first_item || !n_items) return fail(nullptr, A2_EINVAL, "NULL argument");
    if (b < 0 || b + 1 >= (int64_t)s->batch_first.size()) return fail(nullptr, A2_ERANGE, "batch out of range");
    *first_item = s->batch_first[(size_t)b];
    *n_items = s->batch_first[(size_t)b + 1] - s->batch_first[(size_t)b];
    return A2_OK;
}

int a2cid2_sched_item(const a2cid2_sched_t* s, int64_t item, a2cid2_item_info* out) {
    if (!s || !out) return fail(nullptr, A2_EINVAL, "NULL argument");
    if (item < 0 || item >= (int64_t)s->items.size()) return fail(nullptr, A2_ERANGE, "item out of range");
    const a2::SchedItem& it = s->items[(size_t)item];
    *out = a2cid2_item_info{it.a, it.b, it.slot_a, it.slot_b, it.first_op, it.n_ops, it.batch, it.c, it.slot_c, it.d, it.slot_d};
    return A2_OK;
}

int a2cid2_sched_ops(const a2cid2_sched_t* s, int64_t first_op, int64_t n_ops, int64_t* event_index, int32_t* kind) {
    if (!s) return fail(nullptr, A2_EINVAL, "NULL argument");
    if (first_op < 0 || n_ops < 0 || first_op + n_ops > (int64_t)s->ops.size()) return fail(nullptr, A2_ERANGE, "op range out of bounds");
    for (int64_t k = 0; k < n_ops; ++k) {
        if (event_index) event_index[k] = s->ops[(size_t)(first_op + k)].event;
        if (kind) kind[k] = s->ops[(size_t)(first_op + k)].kind;
    }
    return A2_OK;
}

int a2cid2_sched_op_reloads(const a2cid2_sched_t* s, int64_t first_op, int64_t n_ops, int32_t* reload) {
    if (!s || !reload) return fail(nullptr, A2_EINVAL, "NULL argument");
    if (first_op < 0 || n_ops < 0 || first_op + n_ops > (int64_t)s->ops.size()) return fail(nullptr, A2_ERANGE, "op range out of bounds");
    for (int64_t k = 0; k < n_ops; ++k) reload[k] = s->ops[(size_t)(first_op + k)].reload;
    return A2_OK;
}

int a2cid2_sched_t_final(const a2cid2_sched_t* s, double* t_out) {
    if (!s || !t_out) return fail(nullptr, A2_EINVAL, "NULL argument");
    std::memcpy(t_out, s->t_final.data(), sizeof(double) * (size_t)s->n);
    return A2_OK;
}

int a2cid2_sched_stats(const a2cid2_sched_t* s, int64_t first_batch, int64_t n_batches, int64_t d, int32_t elem_bytes_,
                       a2cid2_stats* out) {
    if (!s || !out) return fail(nullptr, A2_EINVAL, "NULL argument");
    const int64_t nb = (int64_t)s->batch_first.size() - 1;
    if (n_batches < 0) n_batches = nb - first_batch;
    if (first_batch < 0 || n_batches < 0 || first_batch + n_batches > nb || d < 0 || elem_bytes_ <= 0)
        return fail(nullptr, A2_ERANGE, "batch range out of bounds");
    a2::schedule_stats(*s, first_batch, first_batch + n_batches, d, elem_bytes_, true, out);
    std::vector<LaunchRange> launches;
    std::vector<int64_t> bf;
    make_launches(*s, launches, bf);
    out->n_launches = bf[(size_t)(first_batch + n_batches)] - bf[(size_t)first_batch];
    return A2_OK;
}

void a2cid2_sched_destroy(a2cid2_sched_t* s) { delete s; }

// ---- graph quantities ----------------------------------------------------------------------------

int a2cid2_graph_chi(int32_t n, int64_t n_edges, const int32_t* ei, const int32_t* ej, const double* lambda, double* chi1,
                     double* chi2) {
    std::string err;
    const int rc = a2::graph_chi(n, n_edges, ei, ej, lambda, chi1, chi2, err);
    if (rc != A2_OK) a2::set_thread_error(err);
    return rc;
}

int a2cid2_prescribe(double chi1, double chi2, int32_t accelerated, double* eta, double* alpha, double* alpha_tilde) {
    if (!eta || !alpha || !alpha_tilde) return fail(nullptr, A2_EINVAL, "NULL output");
    if (!accelerated) {
        *eta = 0.0; *alpha = 0.5; *alpha_tilde = 0.5;
        return A2_OK;
    }
    if (!(chi1 > 0) || !(chi2 > 0) || !std::isfinite(chi1) || !std::isfinite(chi2))
        return fail(nullptr, A2_EINVAL, "chi_1 and chi_2 must be positive and finite");
    *eta = 1.0 / (2.0 * std::sqrt(chi1 * chi2));
    *alpha = 0.5;
    *alpha_tilde = 0.5 * std::sqrt(chi1 / chi2);
    return A2_OK;
}

}  // extern "C"
