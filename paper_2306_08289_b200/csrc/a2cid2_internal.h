// Internal declarations shared by the host scheduler, the kernels' launchers and the C ABI.
#pragma once

#include <cstdint>
#include <cstdlib>
#include <string>
#include <vector>

#include "a2cid2.h"

namespace a2 {

// ---- tuning knobs ---------------------------------------------------------------------------
// The launch shapes (CTAs per SM, vector width, workers per item) are fixed by measurement. A build with
// -DA2_TUNING_KNOBS=1 lets the environment override them for sweeps (A2CID2_EVENT_CTAS_PER_SM,
// A2CID2_EVENT3_CTAS_PER_SM, A2CID2_EVENT4_CTAS_PER_SM, A2CID2_PLAIN_CTAS_PER_SM, A2CID2_PLAIN3_CTAS_PER_SM: resident
// CTAs per SM of the kernel instances; A2CID2_FORCE_128BIT, A2CID2_EVENT4_128BIT: 128-bit accesses;
// A2CID2_ITEM_WORKERS: most workers per chained item). The default build reads none of them.
#ifndef A2_TUNING_KNOBS
#define A2_TUNING_KNOBS 0
#endif
inline const char* tuning_env(const char* name) {
#if A2_TUNING_KNOBS
    return std::getenv(name);
#else
    (void)name;
    return nullptr;
#endif
}

// ---- error text ---------------------------------------------------------------------------
void set_thread_error(const std::string& msg);
const char* thread_error();

// ---- host schedule ------------------------------------------------------------------------
struct SchedOp {
    int64_t event;    // index into the caller's event arrays
    int32_t kind;     // A2_OP_*
    double t;         // event time
    double t_prev_a;  // time the operation's first (or only) worker was last updated before it
    double t_prev_b;  // same for the second worker of a communication
    int32_t reload = -1;  // gradient operations: the row to load into the worker's gradient registers once this
                          // operation has used them (the row of the worker's next gradient operation in the item,
                          // when it differs), or -1
};

constexpr int kMaxItemWorkers = 4;

struct SchedItem {
    int32_t a, b, c, d;  // workers; b, c, d = -1 when absent
    int32_t slot_a, slot_b, slot_c, slot_d;
    int64_t first_op;
    int32_t n_ops;
    int32_t batch;
};

}  // namespace a2

struct a2cid2_sched {
    int32_t n = 0;
    int32_t n_grad_slots = 0;
    uint32_t flags = 0;
    int64_t n_events = 0;
    std::vector<a2::SchedItem> items;  // sorted by batch, creation order inside a batch
    std::vector<a2::SchedOp> ops;      // in item order
    std::vector<int64_t> batch_first;  // items of batch b: [batch_first[b], batch_first[b+1])
    std::vector<double> t_start, t_final;
};

namespace a2 {

// Resident mode (one launch, column tile of the whole population in shared memory).
struct ResEv {  // one event, as the resident kernel reads it (16 bytes)
    int16_t a, b;  // workers (b = -1: gradient event)
    int16_t g;     // index of the gradient row in the chunk's cache, or -1
    int16_t kind;  // A2_OP_GRAD_A or A2_OP_COMM
    float ca, cb;  // mixing coefficients of a and b for this event
};
struct ResChunk {
    int32_t ev_begin, ev_end;  // events of the chunk
    int32_t g_begin, g_count;  // its gradient rows: g_rows[g_begin .. g_begin + g_count)
};
constexpr int kResidentCols = 256;     // columns per tile = threads per CTA
constexpr int kResidentMaxRows = 216;  // 2 n + cache rows, 1 KB of shared memory each
constexpr int kResidentMinCache = 16;

void build_resident_chunks(const a2cid2_sched& s, int capacity, std::vector<ResChunk>& chunks,
                           std::vector<int32_t>& g_rows, std::vector<int32_t>& cache_idx);

// Builds a schedule; returns A2_OK or an error code with the text in `err`.
int build_schedule(int32_t n, int32_t n_grad_slots, const double* t_last, int64_t n_events, const double* times,
                   const int32_t* wi, const int32_t* wj, const int32_t* slot, uint32_t flags,
                   int32_t max_ops_per_item, int32_t max_workers_per_item, a2cid2_sched** out, std::string& err);

// momentum = false counts the rows of the dynamic without x~ (Eq. (baselinedynamic)).
void schedule_stats(const a2cid2_sched& s, int64_t b0, int64_t b1, int64_t d, int32_t elem_bytes, bool momentum,
                    a2cid2_stats* out);

// ---- device descriptors (layout shared by host packing and the event kernel) ---------------
struct DevItem {
    int32_t a, b, c, d, slot_a, slot_b, slot_c, slot_d;
    int32_t op_first;  // relative to the launch's first op
    int32_t op_count;
};

struct DevOp {
    int32_t kind;
    int32_t reload;   // gradient row to fetch into the worker's gradient registers after this operation, or -1
    double t;         // event time
    double t_prev_a;  // last-event time, before this op, of its first (or only) worker
    double t_prev_b;  // of the second worker of a communication
};

constexpr int kMaxItemsPerLaunch = 128;
constexpr int kMaxOpsPerLaunch = 512;
constexpr int kDefaultMaxOpsPerItem = 32;

struct EventLaunch {
    void* x;
    void* xt;
    const void* g;
    int64_t pitch;  // elements
    int64_t d;
    const DevItem* items;  // device
    const DevOp* ops;      // device
    int32_t n_items;
    int32_t n_ops;
    double eta;
    float alpha, alpha_tilde, gamma;
    int32_t variant;
    int32_t dtype;
    int32_t max_workers;  // most workers any item of the launch holds (2, 3 or 4): selects the kernel instance
    int32_t op_base = 0;  // index, in the plan, of the launch's first operation
    bool slice = false;   // column-slice launch: the items may span several batches, each CTA owns a range of columns
    bool has_reloads = false;  // some operation of the launch fetches a gradient row in the middle of its item
    bool round_per_store = false;  // A2_ROUND_PER_STORE: x carried as a two-word value inside an item
};

struct DeviceInfo {
    int sm_count = 0;
    int event_ctas_per_sm[2][2] = {{0, 0}, {0, 0}};  // [storage type][128-bit / 256-bit accesses]
    int event3_ctas_per_sm[2][2] = {{0, 0}, {0, 0}};  // the same for the three-worker instances
    int event4_ctas_per_sm[2] = {0, 0};               // four-worker instances (fp32 rows only): 128-bit / 256-bit
    int plain_ctas_per_sm[2][2] = {{0, 0}, {0, 0}};  // the same for the kernel of the dynamic without x~
    int plain3_ctas_per_sm[2][2] = {{0, 0}, {0, 0}};
    int consensus_ctas_per_sm = 0;
};

// Launchers (kernels.cu). All return a cudaError_t cast to int (0 = success).
int query_device(DeviceInfo* info);
int launch_events(const EventLaunch& L, const DeviceInfo& dev, void* stream);
bool rows_allow_256bit(const void* x, const void* xt, const void* g, int64_t pitch, int32_t dtype);
// Consensus distance. dt (device, n doubles) is NULL for the stored state; partials is device
// scratch of n_partials doubles; out is a device double.
int consensus_grid(const DeviceInfo& dev);
int launch_consensus(const void* x, const void* xt, int64_t pitch, int32_t n, int64_t d, int32_t dtype, double eta,
                     const double* dt, double* partials, int n_partials, double* out, void* stream);

// Resident mode. prepare: items/ops (one op per item, stream order; DevItem.slot_b = cache index) -> ResEv.
struct ResidentLaunch {
    void* x;
    void* xt;
    const void* g;
    int64_t pitch, d;
    int32_t n, dtype, variant;
    double eta;
    float alpha, alpha_tilde, gamma;
    const DevItem* items;    // device, n_events
    const DevOp* ops;        // device, n_events
    ResEv* events;           // device, n_events (written by the prepare kernel)
    const ResChunk* chunks;  // device
    const int32_t* g_rows;   // device
    int32_t n_events, n_chunks, cache_rows;
};
int resident_cache_rows(int32_t n, int32_t n_grad_slots);  // 0: the population does not fit
int launch_resident(const ResidentLaunch& L, const DeviceInfo& dev, void* stream);

// Consensus distance of the stored state with the partial sums in the library's fixed device
// array (no allocation anywhere). out_device is a device double. Returns a cudaError_t as int.
constexpr int kStaticMaxPartials = 4096;
int launch_consensus_static(const void* x, int64_t pitch, int32_t n, int64_t d, int32_t dtype, double* out_device,
                            void* stream, int* n_partials_out);
int64_t consensus_static_max_columns(int32_t dtype);

// ---- spectral (spectral.cpp) -----------------------------------------------------------------
int graph_chi(int32_t n, int64_t n_edges, const int32_t* ei, const int32_t* ej, const double* lambda, double* chi1,
              double* chi2, std::string& err);

}  // namespace a2
