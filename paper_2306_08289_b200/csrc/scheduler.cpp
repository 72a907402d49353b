// Host scheduler: validates a time-sorted event stream and packs it into batches of
// worker-disjoint items that keep every worker's own event order.
//
// Why batches are legal: in Eq. (dynamic) (Sec. 3.2) an event changes only the rows of the
// workers it names, and needs only those rows and their last-event times. Two events on
// disjoint workers therefore commute exactly, and any order that keeps each worker's own
// sequence yields the state of the time-ordered run.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <new>

#include "a2cid2_internal.h"

namespace a2 {

namespace {

struct Pending {
    std::vector<int64_t> events;  // gradient events held back for this worker, in order
    int32_t slot = -1;
};

std::string fmt_event(const char* what, int64_t e) {
    char buf[160];
    std::snprintf(buf, sizeof buf, "event %lld: %s", (long long)e, what);
    return buf;
}

}  // namespace

int build_schedule(int32_t n, int32_t n_grad_slots, const double* t_last, int64_t n_events, const double* times,
                   const int32_t* wi, const int32_t* wj, const int32_t* slot, uint32_t flags,
                   int32_t max_ops_per_item, int32_t max_workers_per_item, a2cid2_sched** out, std::string& err) {
    if (!out) { err = "out is NULL"; return A2_EINVAL; }
    *out = nullptr;
    if (n < 2) { err = "need n >= 2 workers"; return A2_EINVAL; }
    if (n_grad_slots < 0 || n_events < 0) { err = "negative size"; return A2_EINVAL; }
    if (n_events > 0 && (!times || !wi || !wj || !slot)) { err = "event arrays are NULL"; return A2_EINVAL; }
    if (flags & ~uint32_t(A2_SCHED_FUSE | A2_SCHED_RESIDENT | A2_SCHED_CHAIN | A2_SCHED_ROW_PER_OP)) { err = "unknown scheduling flag"; return A2_EINVAL; }
    if (max_workers_per_item <= 0) max_workers_per_item = kMaxItemWorkers;
    if (max_workers_per_item < 2 || max_workers_per_item > kMaxItemWorkers) { err = "an item holds 2 to 4 workers"; return A2_EINVAL; }
    if (max_ops_per_item <= 0) max_ops_per_item = kDefaultMaxOpsPerItem;
    if (max_ops_per_item > kMaxOpsPerLaunch) max_ops_per_item = kMaxOpsPerLaunch;
    const bool resident = (flags & A2_SCHED_RESIDENT) != 0;
    const bool chain = !resident && (flags & A2_SCHED_CHAIN) != 0 && max_ops_per_item >= 2;
    const bool fuse = !resident && ((flags & A2_SCHED_FUSE) != 0 || chain) && max_ops_per_item >= 2;
    const bool row_per_op = fuse && (flags & A2_SCHED_ROW_PER_OP) != 0;  // a worker's gradient row may change inside an item

    a2cid2_sched* s = new (std::nothrow) a2cid2_sched();
    if (!s) { err = "out of host memory"; return A2_ENOMEM; }
    try {
        s->n = n;
        s->n_grad_slots = n_grad_slots;
        s->flags = flags;
        s->n_events = n_events;
        s->t_start.assign((size_t)n, 0.0);
        if (t_last) {
            for (int32_t w = 0; w < n; ++w) {
                if (!std::isfinite(t_last[w])) { err = "non-finite worker time"; delete s; return A2_EINVAL; }
                s->t_start[(size_t)w] = t_last[w];
            }
        }

        // ---- pass 1: validation only (nothing is built from a bad stream) ------------------
        {
            std::vector<double> tcur(s->t_start);
            double prev = -INFINITY;
            for (int64_t e = 0; e < n_events; ++e) {
                const double t = times[e];
                const int32_t i = wi[e], j = wj[e], sl = slot[e];
                if (!std::isfinite(t)) { err = fmt_event("time is not finite", e); delete s; return A2_EINVAL; }
                if (t < prev) { err = fmt_event("times decrease", e); delete s; return A2_EORDER; }
                prev = t;
                if (i < 0 || i >= n) { err = fmt_event("worker index out of range", e); delete s; return A2_ERANGE; }
                if (j == -1) {
                    if (sl < 0 || sl >= n_grad_slots) { err = fmt_event("gradient slot out of range", e); delete s; return A2_ERANGE; }
                    if (t < tcur[(size_t)i]) { err = fmt_event("precedes the worker's last event", e); delete s; return A2_EORDER; }
                    tcur[(size_t)i] = t;
                } else {
                    if (j < 0 || j >= n || j == i) { err = fmt_event("bad pair", e); delete s; return A2_ERANGE; }
                    if (sl != -1) { err = fmt_event("communication event with a gradient slot", e); delete s; return A2_ERANGE; }
                    if (t < tcur[(size_t)i] || t < tcur[(size_t)j]) { err = fmt_event("precedes a worker's last event", e); delete s; return A2_EORDER; }
                    tcur[(size_t)i] = t;
                    tcur[(size_t)j] = t;
                }
            }
        }

        // ---- pass 2: greedy level assignment ------------------------------------------------
        // Items are built in creation order; an item's operations form a linked list because, with
        // A2_SCHED_CHAIN, later events may be appended to an item that is no longer the newest one.
        struct Build {
            SchedItem it;
            int64_t head = -1, tail = -1;  // first and last operation
            int32_t cur_row[kMaxItemWorkers] = {-1, -1, -1, -1};   // gradient row each worker's registers hold at the item's end so far
            int64_t last_gop[kMaxItemWorkers] = {-1, -1, -1, -1};  // each worker's latest gradient operation
        };
        std::vector<Build> items;
        std::vector<SchedOp> ops;      // creation order
        std::vector<int64_t> op_next;  // next operation of the same item, or -1
        items.reserve((size_t)n_events);
        ops.reserve((size_t)n_events);
        op_next.reserve((size_t)n_events);
        std::vector<int32_t> level((size_t)n, 0);      // first batch in which the worker is free
        std::vector<int64_t> last_item((size_t)n, -1);  // chain: the item (of batch level - 1) that holds the worker's latest events
        std::vector<double> tcur(s->t_start);
        std::vector<Pending> pend(fuse ? (size_t)n : 0);

        auto new_item = [&](int32_t a, int32_t b, int32_t batch) -> int64_t {
            Build bd;
            bd.it = SchedItem{a, b, -1, -1, -1, -1, -1, -1, 0, 0, batch};
            items.push_back(bd);
            return (int64_t)items.size() - 1;
        };
        auto add_op = [&](int64_t k, const SchedOp& op) {
            const int64_t o = (int64_t)ops.size();
            ops.push_back(op);
            op_next.push_back(-1);
            Build& bd = items[(size_t)k];
            if (bd.tail >= 0) op_next[(size_t)bd.tail] = o; else bd.head = o;
            bd.tail = o;
            bd.it.n_ops += 1;
        };
        auto local_of = [&](const SchedItem& it, int32_t w) -> int { return it.a == w ? 0 : (it.b == w ? 1 : (it.c == w ? 2 : 3)); };
        auto slot_ref = [&](SchedItem& it, int l) -> int32_t& {
            return l == 0 ? it.slot_a : (l == 1 ? it.slot_b : (l == 2 ? it.slot_c : it.slot_d));
        };
        // can the held-back gradient events of worker w go into item k (which holds w)?
        auto slot_ok = [&](int64_t k, int32_t w) -> bool {
            const Pending& p = pend[(size_t)w];
            if (p.events.empty() || row_per_op) return true;
            SchedItem& it = items[(size_t)k].it;
            const int32_t cur = slot_ref(it, local_of(it, w));
            return cur == -1 || cur == p.slot;
        };
        // append the held-back gradient events of worker w to item k (which holds w)
        auto push_pending = [&](int64_t k, int32_t w) {
            Pending& p = pend[(size_t)w];
            if (p.events.empty()) return;
            const int l = local_of(items[(size_t)k].it, w);
            const int32_t kind = l == 0 ? A2_OP_GRAD_A : (l == 1 ? A2_OP_GRAD_B : (l == 2 ? A2_OP_GRAD_C : A2_OP_GRAD_D));
            for (int64_t e : p.events) {
                Build& bd = items[(size_t)k];
                const int32_t row = slot[e];
                if (bd.cur_row[l] < 0) slot_ref(bd.it, l) = row;  // the worker's first gradient row: read with the state rows
                else if (bd.cur_row[l] != row) ops[(size_t)bd.last_gop[l]].reload = row;  // fetched once the previous one is used
                bd.cur_row[l] = row;
                add_op(k, SchedOp{e, kind, times[e], tcur[(size_t)w], 0.0});
                items[(size_t)k].last_gop[l] = (int64_t)ops.size() - 1;
                tcur[(size_t)w] = times[e];
            }
            p.events.clear();
            p.slot = -1;
        };
        // the communication of event e between workers i and j, both held by item k
        auto push_comm = [&](int64_t k, int64_t e, int32_t i, int32_t j) {
            const SchedItem& it = items[(size_t)k].it;
            int li = local_of(it, i), lj = local_of(it, j);
            int32_t wa = i, wb = j;
            if (li > lj) { std::swap(li, lj); std::swap(wa, wb); }  // the update is symmetric in the two workers
            static const int32_t kPair[4][4] = {{-1, A2_OP_COMM, A2_OP_COMM_AC, A2_OP_COMM_AD},
                                                {-1, -1, A2_OP_COMM_BC, A2_OP_COMM_BD},
                                                {-1, -1, -1, A2_OP_COMM_CD},
                                                {-1, -1, -1, -1}};
            const int32_t kind = kPair[li][lj];
            add_op(k, SchedOp{e, kind, times[e], tcur[(size_t)wa], tcur[(size_t)wb]});
            tcur[(size_t)i] = times[e];
            tcur[(size_t)j] = times[e];
        };
        auto flush = [&](int32_t w) {  // the worker's held-back gradient events leave the queue
            Pending& p = pend[(size_t)w];
            if (p.events.empty()) return;
            const int64_t kl = chain ? last_item[(size_t)w] : -1;
            if (kl >= 0 && slot_ok(kl, w) && items[(size_t)kl].it.n_ops + (int64_t)p.events.size() <= max_ops_per_item) {
                push_pending(kl, w);  // the item that already holds the worker's rows takes them
                return;
            }
            const int64_t k = new_item(w, -1, level[(size_t)w]);
            push_pending(k, w);
            last_item[(size_t)w] = k;
            level[(size_t)w] += 1;
        };

        for (int64_t e = 0; e < n_events; ++e) {
            const int32_t i = wi[e], j = wj[e];
            if (j == -1) {
                if (fuse) {
                    Pending& p = pend[(size_t)i];
                    if (!p.events.empty() && ((!row_per_op && p.slot != slot[e]) || (int32_t)p.events.size() >= max_ops_per_item - 1)) flush(i);
                    p.slot = slot[e];
                    p.events.push_back(e);
                } else {
                    const int64_t k = new_item(i, -1, level[(size_t)i]);
                    items[(size_t)k].it.slot_a = slot[e];
                    add_op(k, SchedOp{e, A2_OP_GRAD_A, times[e], tcur[(size_t)i], 0.0});
                    tcur[(size_t)i] = times[e];
                    level[(size_t)i] += 1;
                }
                continue;
            }
            if (chain) {
                const int64_t need = (int64_t)pend[(size_t)i].events.size() + (int64_t)pend[(size_t)j].events.size() + 1;
                const int64_t ki = last_item[(size_t)i], kj = last_item[(size_t)j];
                // (1) both workers' rows are already together in one item: the event costs no row at all
                if (ki >= 0 && ki == kj && slot_ok(ki, i) && slot_ok(ki, j) &&
                    items[(size_t)ki].it.n_ops + need <= max_ops_per_item) {
                    push_pending(ki, i);
                    push_pending(ki, j);
                    push_comm(ki, e, i, j);
                    continue;
                }
                // (2) one worker is free earlier than the other: it joins the other's latest item as one more
                // worker of that item, so the other's rows are not stored and read again
                if (level[(size_t)i] != level[(size_t)j]) {
                    const int32_t hi = level[(size_t)i] > level[(size_t)j] ? i : j, lo = hi == i ? j : i;
                    const int64_t kh = last_item[(size_t)hi];
                    const int held = kh < 0 ? 0 : (items[(size_t)kh].it.b < 0 ? 1 : (items[(size_t)kh].it.c < 0 ? 2 : (items[(size_t)kh].it.d < 0 ? 3 : 4)));
                    if (kh >= 0 && held + 1 <= max_workers_per_item && slot_ok(kh, hi) &&
                        items[(size_t)kh].it.n_ops + need <= max_ops_per_item) {
                        SchedItem& it = items[(size_t)kh].it;
                        if (it.b < 0) it.b = lo; else if (it.c < 0) it.c = lo; else it.d = lo;
                        push_pending(kh, i);
                        push_pending(kh, j);
                        push_comm(kh, e, i, j);
                        level[(size_t)lo] = level[(size_t)hi];
                        last_item[(size_t)lo] = kh;
                        continue;
                    }
                }
            }
            if (fuse) {
                Pending& pi = pend[(size_t)i];
                Pending& pj = pend[(size_t)j];
                if ((int64_t)pi.events.size() + (int64_t)pj.events.size() + 1 > max_ops_per_item) {
                    // too long for one item: spill the longer side first
                    if (pi.events.size() >= pj.events.size()) flush(i); else flush(j);
                    if ((int64_t)pi.events.size() + (int64_t)pj.events.size() + 1 > max_ops_per_item) {
                        flush(i);
                        flush(j);
                    }
                }
            }
            const int32_t lv = std::max(level[(size_t)i], level[(size_t)j]);
            const int64_t k = new_item(i, j, lv);
            if (fuse) {
                push_pending(k, i);
                push_pending(k, j);
            }
            push_comm(k, e, i, j);
            level[(size_t)i] = lv + 1;
            level[(size_t)j] = lv + 1;
            last_item[(size_t)i] = k;
            last_item[(size_t)j] = k;
        }
        if (fuse) for (int32_t w = 0; w < n; ++w) flush(w);
        if (resident)  // one batch, every event in stream order (items were created in that order)
            for (Build& bd : items) bd.it.batch = 0;

        // ---- order items by batch (stable) and lay the ops out in item order ----------------
        int32_t n_batches = 0;
        for (const Build& bd : items) n_batches = std::max(n_batches, bd.it.batch + 1);
        s->batch_first.assign((size_t)n_batches + 1, 0);
        for (const Build& bd : items) s->batch_first[(size_t)bd.it.batch + 1] += 1;
        for (int32_t b = 0; b < n_batches; ++b) s->batch_first[(size_t)b + 1] += s->batch_first[(size_t)b];
        std::vector<int64_t> cursor(s->batch_first.begin(), s->batch_first.end() - 1);
        s->items.resize(items.size());
        std::vector<int64_t> heads(items.size());
        for (const Build& bd : items) {
            const int64_t dst = cursor[(size_t)bd.it.batch]++;
            s->items[(size_t)dst] = bd.it;
            heads[(size_t)dst] = bd.head;
        }
        s->ops.reserve(ops.size());
        for (size_t k = 0; k < s->items.size(); ++k) {
            s->items[k].first_op = (int64_t)s->ops.size();
            for (int64_t o = heads[k]; o >= 0; o = op_next[(size_t)o]) s->ops.push_back(ops[(size_t)o]);
        }
        s->t_final = tcur;
    } catch (const std::bad_alloc&) {
        delete s;
        err = "out of host memory";
        return A2_ENOMEM;
    }
    *out = s;
    return A2_OK;
}

// Resident mode: cut the stream into chunks whose distinct gradient rows fit `capacity` cache rows.
// Inside a chunk a gradient row keeps the cache index it was given at first use.
void build_resident_chunks(const a2cid2_sched& s, int capacity, std::vector<ResChunk>& chunks,
                           std::vector<int32_t>& g_rows, std::vector<int32_t>& cache_idx) {
    chunks.clear();
    g_rows.clear();
    cache_idx.assign(s.items.size(), -1);
    std::vector<int32_t> where((size_t)std::max(1, s.n_grad_slots), -1);  // slot -> cache index in the open chunk
    ResChunk cur{0, 0, 0, 0};
    auto close = [&](int32_t ev_end) {
        cur.ev_end = ev_end;
        if (cur.ev_end > cur.ev_begin) chunks.push_back(cur);
        for (int32_t k = cur.g_begin; k < cur.g_begin + cur.g_count; ++k) where[(size_t)g_rows[(size_t)k]] = -1;
        cur = ResChunk{ev_end, ev_end, (int32_t)g_rows.size(), 0};
    };
    for (size_t e = 0; e < s.items.size(); ++e) {
        const int32_t slot = s.items[e].slot_a;
        if (slot < 0) continue;
        if (where[(size_t)slot] < 0) {
            if (cur.g_count == capacity) close((int32_t)e);
            where[(size_t)slot] = cur.g_count;
            g_rows.push_back(slot);
            cur.g_count += 1;
        }
        cache_idx[e] = where[(size_t)slot];
    }
    close((int32_t)s.items.size());
}

void schedule_stats(const a2cid2_sched& s, int64_t b0, int64_t b1, int64_t d, int32_t elem_bytes, bool momentum,
                    a2cid2_stats* out) {
    a2cid2_stats st{};
    const int64_t i0 = s.batch_first[(size_t)b0], i1 = s.batch_first[(size_t)b1];
    int64_t rows_moved = 0, rows_single = 0;
    for (int64_t k = i0; k < i1; ++k) {
        const SchedItem& it = s.items[(size_t)k];
        const int64_t per_worker = momentum ? 2 : 1;  // x and x~, or x alone
        const int64_t state_rows = (1 + (it.b >= 0 ? 1 : 0) + (it.c >= 0 ? 1 : 0) + (it.d >= 0 ? 1 : 0)) * per_worker;
        bool touches_state = momentum;  // without x~ a mixing-only item moves nothing
        for (int32_t o = 0; o < it.n_ops && !touches_state; ++o)
            touches_state = s.ops[(size_t)(it.first_op + o)].kind != A2_OP_MIX_A;
        if (touches_state)
            rows_moved += 2 * state_rows + (it.slot_a >= 0 ? 1 : 0) + (it.slot_b >= 0 ? 1 : 0) + (it.slot_c >= 0 ? 1 : 0) +
                          (it.slot_d >= 0 ? 1 : 0);
        for (int32_t o = 0; o < it.n_ops; ++o) {
            if (s.ops[(size_t)(it.first_op + o)].reload >= 0) rows_moved += 1;  // a gradient row fetched inside the item
            const int32_t kind = s.ops[(size_t)(it.first_op + o)].kind;
            if (kind == A2_OP_COMM || kind == A2_OP_COMM_AC || kind == A2_OP_COMM_BC || kind == A2_OP_COMM_AD ||
                kind == A2_OP_COMM_BD || kind == A2_OP_COMM_CD) { st.n_comm += 1; rows_single += momentum ? 8 : 4; }
            else if (kind == A2_OP_MIX_A) { rows_single += momentum ? 4 : 0; }
            else { st.n_grad += 1; rows_single += momentum ? 5 : 3; }
        }
    }
    st.n_events = st.n_comm + st.n_grad;
    st.n_batches = b1 - b0;
    st.n_items = i1 - i0;
    st.bytes_moved = rows_moved * d * elem_bytes;
    st.bytes_one_by_one = rows_single * d * elem_bytes;
    *out = st;
}

}  // namespace a2
