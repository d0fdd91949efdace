// pie_pool: the HBM + pinned-host block pools, streams and events around the mapping table, the swap
// and attention entry points, the per-layer decode loop, the controller tick and the C ABI.
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstddef>
#include <cstdio>
#include <cstring>
#include <deque>
#include <new>
#include <vector>

#include "pie_kernels.h"
#include "pie_table.h"

namespace {

thread_local int g_last_cuda_error = 0;

constexpr int EV_RING = 512;       // events per queue: ticket t uses slot t % EV_RING
constexpr int LIST_EVENTS = 512;   // events guarding regions of the id-list ring
constexpr int TIMING_RING = 4;     // the host may enqueue at most this many steps ahead of their evaluation
constexpr int64_t AUTO_COPY_ENGINE_RUN_BYTES = 1 << 20;  // AUTO: copy engine when runs average >= 1 MiB ...
constexpr int64_t AUTO_COPY_ENGINE_MAX_RUNS = 8;         // ... or when the list is at most this many runs
constexpr int IO_GROUP_LAYERS = 4;   // pie_decode_step_host moves inputs and results in groups of this many layers
constexpr int64_t PATCH_DMA_MAX_RUNS = 16;               // table entries by small copies up to this many runs of ids, else a kernel

#define PIE_CUDA(call)                                  \
    do {                                                \
        cudaError_t e__ = (call);                       \
        if (e__ != cudaSuccess) {                       \
            g_last_cuda_error = (int)e__;               \
            return PIE_ERR_CUDA;                        \
        }                                               \
    } while (0)

struct LayerEvents {
    // Copy streams: timing events at the start of a list (in0, out0, owned) and its ticket's event at the end (in1,
    // out1: valid for EV_RING tickets).  The compute stream carries no timing events at all - a record there costs
    // 2-3 us between two kernels; the attention kernel notes the GPU timer itself (stamps, below).  For the per-layer
    // timeline (timing = 2) one timing event per step on the compute stream, recorded right before the step's first
    // attention kernel, ties the copy streams' events to the stamps (to within the few us between that record and
    // the kernel's start).
    cudaEvent_t in0 = nullptr, in1 = nullptr, out0 = nullptr, out1 = nullptr;
    bool has_in = false, has_out = false, has_compute = false;
    bool stream_wait = false;   // the layer's attention call made the compute stream wait for a copy's event
};
// per layer of a step: GPU-timer stamps in mapped pinned memory
// START: CTA 0 begins its main work (after the dependency wait), END: the last CTA leaves, WAIT: ns CTA 0's producer
// spent in the presence wait, TOKENS: the batch's context tokens
enum { STAMP_START = 0, STAMP_END = 1, STAMP_WAIT = 2, STAMP_TOKENS = 3, STAMP_WORDS = 4 };
constexpr int MAX_GROUP_LAYERS = 8;  // layers whose swap lists are issued together (pie_set_lookahead)

struct ListRecord {
    int64_t start, end;
    int ev;          // index into list_events, or -1: guarded by a ticket of a queue (its event is recorded by the caller)
    int queue;
    int64_t ticket;
};

// One swap list after phase 1 of the table update (Section 3.2): destination slots chosen and recorded, source slots
// released under the list's ticket; nothing enqueued yet.
struct SwapList {
    int32_t layer = 0;
    int64_t ticket = 0, n_moved = 0, n_elided = 0;
    std::vector<int32_t> moved, src, dst;
    std::vector<uint8_t> elide;
    int64_t waits[4] = {0, 0, 0, 0};
};

}  // namespace

struct pie_pool {
    pie_pool_config cfg{};
    int64_t block_bytes = 0;
    int kv_fp8 = 0;                       // blocks hold E4M3 bytes (cfg.kv_format)
    float k_scale = 1.f, v_scale = 1.f;   // a stored byte stands for decode(byte) * scale
    pie::Table *table = nullptr;
    uint8_t *gpu_base = nullptr, *host_base = nullptr;
    bool own_gpu = false, own_host = false, own_streams = false;
    cudaStream_t stream[4] = {nullptr, nullptr, nullptr, nullptr};  // indexed by queue id
    cudaEvent_t ticket_ev[4][EV_RING] = {};
    // Marks on the compute stream come from two rings of events (compute_mark picks per record).
    // A record without a time stamp is ~2.5 us cheaper between two kernels, but when another stream waits on such an
    // event the recording stream loses ~5 us instead (measured on this part and driver): so plain events while
    // nothing is being swapped, time-stamped ones while swap lists, which wait on compute tickets, are in flight.
    cudaEvent_t compute_ev_plain[EV_RING] = {}, compute_ev_stamped[EV_RING] = {};
    // An event on the compute stream between two layers costs every layer a few microseconds (and keeps the next
    // attention kernel from being launched as a dependent of the previous one), so compute tickets get an event only
    // where somebody has to wait for one: a mark is recorded at the stream's tail and covers every ticket enqueued so far.
    struct ComputeMark {
        int64_t ticket;
        cudaEvent_t ev;
    };
    // Where the driver offers stream waits by value, the copy streams do not need a mark either: the attention kernel's
    // last CTA stores its call's ticket in a device word and a copy stream waits until the word has reached the ticket
    // it needs.  A mark between two layers serialises the next kernel's launch behind it, and that launch is slow while
    // swap lists are crossing the host link; the word costs the compute stream nothing.
    unsigned long long *done_dev = nullptr;   // newest compute ticket whose attention kernel has completed
    int64_t last_attn_ticket = 0;             // newest compute ticket an attention kernel will store there
    CUresult (*wait_value64)(CUstream, CUdeviceptr, cuuint64_t, unsigned int) = nullptr;
    std::deque<ComputeMark> compute_marks;   // recorded, not yet known complete; tickets ascending
    int compute_ev_next = 0;                 // next slot of the two event rings
    int64_t compute_marked = 0;              // newest compute ticket that a recorded mark covers
    // Presence wait inside the attention kernel: per layer a device word that the copy-in stream sets to a list's ticket
    // (a small copy behind the list's blocks and table entries).  Lists moved or patched by an SM kernel are waited for
    // with a stream-level event wait instead: a kernel that polls while it owns the SMs must not wait for another kernel.
    unsigned long long *arrive_dev = nullptr;   // [n_layers]
    std::vector<int64_t> layer_in_sm;           // per layer: newest in-ticket that involved an SM kernel
    std::vector<int64_t> layer_in_last;         // per layer: newest in-ticket whose list sets the layer's arrival word
    // Swap lists are issued for a group of consecutive layers at a time: while a group computes, the next group's shares
    // arrive and the previous group's leave; one mark on the compute stream per group.
    int32_t group_setting = 0;                  // 0: chosen per group from the staging the GPU pool can afford
    int32_t group_first = 0, group_len = 0;     // the group in progress (group_len 0: none)
    std::vector<int32_t> group_done;            // its layers that have computed and whose share has yet to go out
    int32_t group_mode = PIE_MODE_AUTO;
    int64_t last_swap_step = -2;   // the step in which the newest swap list was issued
    int64_t recorded[4] = {0, 0, 0, 0};  // newest ticket of each queue whose event has been recorded
    int32_t *slot_table_dev = nullptr;  // [L][NB]
    // id lists: pinned ring + device mirror at the same offsets
    int32_t *list_host = nullptr, *list_dev = nullptr;
    int64_t list_words = 0, list_head = 0;
    std::deque<ListRecord> list_live;
    cudaEvent_t list_events[LIST_EVENTS] = {};
    int list_ev_next = 0;
    // device status word (mapped pinned memory)
    int32_t *status_host = nullptr, *status_dev = nullptr;
    uint64_t *stamps_host = nullptr, *stamps_dev = nullptr;  // [TIMING_RING][n_layers][STAMP_WORDS]: pinned copy, device original
    uint64_t free_step_gap_ns = 0;   // smallest gap between two layers' attention kernels in the newest step without swaps
    uint64_t prev_step_end = 0;   // GPU-timer stamp of the end of the last layer of the newest evaluated step
    int64_t prev_step_id = -1;
    // attention
    pie::AttnScratch scratch{};
    CUtensorMap map3d{}, map2d{};
    CUtensorMap map_prefill{};   // the pool's K and V rows as 16-row tiles (chunked-prefill attention; 16-bit pools)
    bool prefill_ready = false;
    int use3d = 0, attn_grid = 0, n_sms = 0;
    // decode-step staging (device copies of host inputs)
    void *stage_q = nullptr, *stage_out = nullptr, *stage_k = nullptr, *stage_v = nullptr;
    int32_t *stage_bt = nullptr, *stage_ctx = nullptr;
    int64_t stage_q_bytes = 0, stage_kv_bytes = 0, stage_bt_words = 0;
    // policy / controller
    int ratio_mode = 0;  // 0 unset (keep the caller's sets), 1 fixed, 2 adaptive
    double ratio = 0.0;
    double ctrl_state[16] = {};
    pie_governor *governor = nullptr;   // throughput records (pie_report_throughput); created at the first report
    double ratio_cap = 1.0;
    double ctrl_step = 0.0;  // 0: one layer's worth, 1 / n_layers
    int32_t lookahead = 1;   // how many layers ahead the decode loop prefetches (Section 3.4.2 uses 1)
    bool poll_hold = false;  // a decode step is polling once per layer: nested calls skip theirs
    std::vector<int64_t> home_count;  // per layer: units whose home is the host
    std::vector<std::vector<int32_t>> home_list;  // per layer: ids the planner looks at (see candidate_ids)
    std::vector<uint8_t> home_dirty;              // per layer: home_list must be rebuilt
    // whole-layer protocol (Section 3.3): when set, pie_decode_step moves whole layers as the scheduler says
    double layer_ctrl_state[4] = {};   // whole-layer adaptive rule (pie_layer_controller_decide)
    double violation_trigger = 0.0;    // share of next-token prefetches that triggers an increase (0: the rule's default)
    int64_t step_prefetch[TIMING_RING][2] = {};   // per step set: swap-in lists started, of which for the next token
    int32_t fifo_cpu_layers = 0;       // whole-layer mode: m, the layers that live on the CPU (cpu_regions - 2)
    pie::Fifo *fifo = nullptr;
    int64_t fifo_ticket[3] = {0, 0, 0};        // ticket of the layer swap in flight, per queue (0 = none)
    std::vector<int32_t> fifo_log;             // {step, layer starting, swap-out started or -1, swap-in started or -1} x n
    // timing
    // per-step event sets: step k uses set k % TIMING_RING; a set is evaluated once, in step order, when complete
    std::vector<LayerEvents> lev[TIMING_RING];
    int64_t lev_step[TIMING_RING] = {};      // which step a set holds (0 = none)
    bool lev_done[TIMING_RING] = {};         // already evaluated
    bool lev_closed[TIMING_RING] = {};       // the step's last compute ticket has its mark (or needs none)
    cudaEvent_t lev_anchor[TIMING_RING] = {};   // timing = 2: recorded on the compute stream before the step's first attention kernel
    bool lev_anchored[TIMING_RING] = {};
    cudaEvent_t lev_last[TIMING_RING][4] = {};  // the set's newest event on each queue's stream (its streams complete in order)
    cudaStream_t aux_stream = nullptr;          // brings a step's stamps to the host without touching the compute stream
    cudaEvent_t lev_close_ev[TIMING_RING] = {}; // recorded there behind the copy
    cudaEvent_t step_end_ev[TIMING_RING] = {};  // recorded there once a step's last attention kernel has completed
    int64_t step_end_of[TIMING_RING] = {};      // ... the step each of them stands for (0 = none)
    int64_t step_end_ticket = 0;                // the compute ticket the newest of them waits for
    int32_t run_ahead = 2;                      // steps the host may be ahead of the GPU (pie_set_run_ahead)
    int64_t step = 0;
    double base_ms_per_token = 0.0;  // attention time per context token measured on steps without swap traffic
    double free_contrast = -1.0;     // on swap-free steps: the contrast of the layers' four-layer mean times (see evaluate_step_set)
    std::vector<float> timeline;     // last evaluated step: [L][7] ms from the step's first event (-1 = not recorded)
    pie_stats stats{};
    // scratch vectors
    std::vector<int32_t> v_moved, v_src, v_dst, v_in, v_out;
    SwapList one_list;                  // the list of a single swap call
    // split-K merge left to the next attention call of the decode step (its kernel merges in the tail of its launch)
    bool auto_split = false;            // the configuration left the split-K chunk to the library
    struct Deferred {
        bool on = false;
        void *out = nullptr;
        const int32_t *ctx = nullptr;
        int parity = 0;
        int32_t n_seqs = 0, max_blocks = 0, split = 0;
    } deferred;
    std::vector<SwapList> group_lists;  // the lists of a group of layers (decode loop)
    std::vector<uint8_t> v_elide;
    cudaStream_t io_stream[2] = {nullptr, nullptr};  // pie_decode_step_host: inputs up / results down
    unsigned long long *io_arrive_dev = nullptr;     // counts the groups of layers whose inputs have arrived (set by io_stream[0])
    unsigned long long io_groups_up = 0;             // ... as issued by the host
    unsigned long long inputs_need = 0;              // what the next attention call's kernel has to wait for (0: nothing)
    std::vector<int32_t> v_plan_in, v_plan_out;  // one layer's plan inside the decode loop
    std::vector<int32_t> append_ids;  // blocks the coming appends write (pie_declare_append_blocks)
    bool append_declared = false;
    int sticky = PIE_OK;
};

namespace {

// Phase 2 of the table update (Section 3.2): learn which copies and attention calls have completed.  While a
// decode step holds the poll (one forced poll per layer there), the calls inside it skip their own.
int poll(pie_pool *p, bool force = false) {
    if (p->poll_hold && !force) return PIE_OK;
    {
        int64_t d = p->table->done(PIE_Q_COMPUTE);
        while (!p->compute_marks.empty()) {
            cudaError_t e = cudaEventQuery(p->compute_marks.front().ev);
            if (e == cudaErrorNotReady) break;
            if (e != cudaSuccess) {
                g_last_cuda_error = (int)e;
                p->sticky = PIE_ERR_CUDA;
                return PIE_ERR_CUDA;
            }
            d = std::max(d, p->compute_marks.front().ticket);
            p->compute_marks.pop_front();
        }
        if (d > p->table->done(PIE_Q_COMPUTE)) p->table->confirm(PIE_Q_COMPUTE, d);
    }
    for (int q = 1; q <= 2; ++q) {
        int64_t d = p->table->done(q);
        const int64_t issued = p->recorded[q];  // a ticket whose event is not recorded yet cannot be queried
        while (d < issued) {
            cudaError_t e = cudaEventQuery(p->ticket_ev[q][(d + 1) % EV_RING]);
            if (e == cudaSuccess) ++d;
            else if (e == cudaErrorNotReady) break;
            else {
                g_last_cuda_error = (int)e;
                p->sticky = PIE_ERR_CUDA;
                return PIE_ERR_CUDA;
            }
        }
        if (d > p->table->done(q)) p->table->confirm(q, d);
    }
    return PIE_OK;
}

// Record a mark at the compute stream's tail: it covers every compute ticket enqueued so far.
int push_mark(pie_pool *p, cudaEvent_t *ev) {
    if ((int)p->compute_marks.size() >= EV_RING - 1) {  // the ring is full: its oldest mark must complete first
        PIE_CUDA(cudaEventSynchronize(p->compute_marks.front().ev));
        int st = poll(p, true);
        if (st != PIE_OK) return st;
    }
    const int slot = p->compute_ev_next;
    p->compute_ev_next = (slot + 1) % EV_RING;
    // (a time-stamped event is the cheaper one for the recording stream when other streams wait on it)
    cudaEvent_t e = p->last_swap_step >= p->step - 1 ? p->compute_ev_stamped[slot] : p->compute_ev_plain[slot];
    PIE_CUDA(cudaEventRecord(e, p->stream[PIE_Q_COMPUTE]));
    p->compute_marked = p->recorded[PIE_Q_COMPUTE];
    p->compute_marks.push_back({p->compute_marked, e});
    *ev = e;
    return PIE_OK;
}

// The mark that covers compute ticket t: the oldest recorded one at or after it; recorded now, at the stream's tail,
// if there is none yet.  *ev stays null when the ticket is already known complete.
int compute_mark(pie_pool *p, int64_t t, cudaEvent_t *ev) {
    *ev = nullptr;
    if (t <= 0 || t <= p->table->done(PIE_Q_COMPUTE)) return PIE_OK;
    if (t > p->compute_marked) return push_mark(p, ev);
    for (const pie_pool::ComputeMark &m : p->compute_marks)
        if (m.ticket >= t) {
            *ev = m.ev;
            break;
        }
    return PIE_OK;
}

// make `stream` wait for ticket t of queue q (no-op if already known complete)
int wait_ticket(pie_pool *p, cudaStream_t stream, int q, int64_t t) {
    if (t <= 0 || t <= p->table->done(q)) return PIE_OK;
    if (q == PIE_Q_COMPUTE && p->wait_value64 && t <= p->last_attn_ticket && stream != p->stream[PIE_Q_COMPUTE]) {
        if (p->wait_value64((CUstream)stream, (CUdeviceptr)(uintptr_t)p->done_dev, (cuuint64_t)t, CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) {
            g_last_cuda_error = (int)cudaErrorUnknown;
            return PIE_ERR_CUDA;
        }
        return PIE_OK;
    }
    if (q == PIE_Q_COMPUTE) {
        cudaEvent_t ev = nullptr;
        int st = compute_mark(p, t, &ev);
        if (st != PIE_OK) return st;
        if (ev) PIE_CUDA(cudaStreamWaitEvent(stream, ev, 0));
        return PIE_OK;
    }
    PIE_CUDA(cudaStreamWaitEvent(stream, p->ticket_ev[q][t % EV_RING], 0));
    return PIE_OK;
}

// before ticket t of queue q records its event: the slot's previous user (t - EV_RING) must be done
int reserve_ticket_event(pie_pool *p, int q, int64_t t) {
    if (q == PIE_Q_COMPUTE) return PIE_OK;  // compute tickets share marks (compute_mark)
    const int64_t prev = t - EV_RING;
    if (prev > 0 && prev > p->table->done(q)) {
        PIE_CUDA(cudaEventSynchronize(p->ticket_ev[q][prev % EV_RING]));
        poll(p, true);
    }
    return PIE_OK;
}

int record_ticket(pie_pool *p, int q, int64_t t) {
    if (q == PIE_Q_COMPUTE) {  // enqueued; an event follows only if somebody has to wait for it (compute_mark)
        p->recorded[q] = t;
        return PIE_OK;
    }
    PIE_CUDA(cudaEventRecord(p->ticket_ev[q][t % EV_RING], p->stream[q]));
    p->recorded[q] = t;
    return PIE_OK;
}

// reserve `words` int32 in the list ring; waits (bounded by the GPU finishing earlier work) if the ring is full
int list_alloc(pie_pool *p, int64_t words, int64_t *offset) {
    words = (words + 3) & ~int64_t(3);  // 16-byte granules
    if (words > p->list_words) return PIE_ERR_INVALID;
    if (p->list_head + words > p->list_words) p->list_head = 0;
    const int64_t a = p->list_head, b = a + words;
    auto consumed = [&](const ListRecord &r) {
        if (r.ev < 0) return r.ticket <= p->table->done(r.queue);  // as of the last poll: no driver call
        return cudaEventQuery(p->list_events[r.ev]) == cudaSuccess;
    };
    auto wait_for = [&](const ListRecord &r) {
        return cudaEventSynchronize(r.ev < 0 ? p->ticket_ev[r.queue][r.ticket % EV_RING] : p->list_events[r.ev]);
    };
    while (!p->list_live.empty() && consumed(p->list_live.front())) p->list_live.pop_front();
    for (;;) {
        bool clash = false;
        for (size_t i = 0; i < p->list_live.size(); ++i) {
            const ListRecord r = p->list_live[i];
            if (r.start < b && a < r.end) {
                if (!consumed(r)) PIE_CUDA(wait_for(r));
                p->list_live.erase(p->list_live.begin() + (long)i);
                clash = true;
                break;
            }
        }
        if (!clash) break;
    }
    if ((int)p->list_live.size() >= LIST_EVENTS - 1) {
        PIE_CUDA(wait_for(p->list_live.front()));
        p->list_live.pop_front();
    }
    *offset = a;
    p->list_head = b;
    return PIE_OK;
}

// the list at `offset` is consumed by work already enqueued on `stream`: guard it with an event
int list_commit(pie_pool *p, int64_t offset, int64_t words, cudaStream_t stream) {
    words = (words + 3) & ~int64_t(3);
    const int ev = p->list_ev_next;
    p->list_ev_next = (p->list_ev_next + 1) % LIST_EVENTS;
    PIE_CUDA(cudaEventRecord(p->list_events[ev], stream));
    p->list_live.push_back({offset, offset + words, ev, 0, 0});
    return PIE_OK;
}

// the same for a list consumed by work that belongs to ticket t of queue q: the ticket's event, which the caller
// records right after that work, guards the list and no event of its own is needed
void list_commit_ticket(pie_pool *p, int64_t offset, int64_t words, int q, int64_t t) {
    words = (words + 3) & ~int64_t(3);
    p->list_live.push_back({offset, offset + words, -1, q, t});
}

int check_status_word(pie_pool *p) {
    volatile int32_t *w = p->status_host;  // [0] missing unit, [1] context too long, [2] wait timed out
    if (w[0] == 0 && w[1] == 0 && w[2] == 0) return PIE_OK;
    const int st = w[2] ? PIE_ERR_TIMEOUT : w[0] ? PIE_ERR_NOT_RESIDENT : PIE_ERR_INVALID;
    w[0] = w[1] = w[2] = 0;
    return st;
}

LayerEvents *timing_slot(pie_pool *p, int32_t layer) {
    if (!p->cfg.timing) return nullptr;
    return &p->lev[p->step % TIMING_RING][(size_t)layer];
}

// device-visible address of one stamp of the current step's set (nullptr with timing off)
uint64_t *stamp_dev(pie_pool *p, int32_t layer, int which) {
    if (!p->cfg.timing) return nullptr;
    return p->stamps_dev + ((size_t)(p->step % TIMING_RING) * (size_t)p->cfg.n_layers + (size_t)layer) * STAMP_WORDS + which;
}

// ---- one swap call ------------------------------------------------------------------------------------
// elide (optional): pairs flagged 1 move no bytes (a kept, unwritten host copy); they still get their table entry
// patched, and they force the copy-engine path: the gather/scatter kernel takes the whole list.
// arrive (optional, device): behind the list's copies and table entries the ticket is stored there by one small copy -
// the word the layer's attention kernel waits for; *used_sm tells whether an SM kernel moved or patched the list.
int do_copies(pie_pool *p, int dir_queue, const int32_t *src, const int32_t *dst, int64_t n, const int32_t *blocks,
              int32_t *slot_table_row, int mode, cudaStream_t stream, int64_t ticket = 0, const uint8_t *elide = nullptr,
              unsigned long long *arrive = nullptr, bool *used_sm = nullptr) {
    // dir_queue PIE_Q_IN: host -> GPU; PIE_Q_OUT: GPU -> host
    const uint8_t *src_pool = dir_queue == PIE_Q_IN ? p->host_base : p->gpu_base;
    uint8_t *dst_pool = dir_queue == PIE_Q_IN ? p->gpu_base : p->host_base;
    const int64_t BB = p->block_bytes;
    bool any_elided = false;
    if (elide)
        for (int64_t i = 0; i < n && !any_elided; ++i) any_elided = elide[i] != 0;
    if (!any_elided) elide = nullptr;
    if (elide) mode = PIE_MODE_COPY_ENGINE;
    if (mode == PIE_MODE_AUTO) {
        int64_t runs = 1;
        for (int64_t i = 1; i < n; ++i)
            if (src[i] != src[i - 1] + 1 || dst[i] != dst[i - 1] + 1) ++runs;
        // copy engine for long runs or few copies (no SM or L2 footprint next to attention); the bulk-copy kernel for
        // scattered lists, where one cudaMemcpyAsync per piece is bound by the call rate (~2-5 us each) and every
        // separate device-to-host copy costs a concurrent attention kernel a fixed 1-2 % (measured: 21 pieces of
        // 256 KiB per list by copy engine cost 18 %, by kernel far less).  The bulk kernel moves scattered lists at
        // the same rate as the load/store kernel and costs the attention a third of what that one does.
        mode = ((n * BB) / runs >= AUTO_COPY_ENGINE_RUN_BYTES || runs <= AUTO_COPY_ENGINE_MAX_RUNS) ? PIE_MODE_COPY_ENGINE
                                                                                                   : PIE_MODE_KERNEL_BULK;
    }
    // Table entries after copy-engine copies.  A patch kernel on a copy stream, launched while the persistent
    // attention grid owns the SMs, was measured to lengthen the gap between two attention launches, and it puts an
    // SM-side kernel on the path of the ticket the next layer waits for.  When the moved ids form a few runs of
    // consecutive blocks (the usual case: lists are in ascending id), the new entries are written to the pinned list
    // ring instead and one small host-to-device copy per run puts them into the layer's row: no SM is involved.
    bool dma_patch = false;
    if (mode == PIE_MODE_COPY_ENGINE && slot_table_row != nullptr && blocks != nullptr) {
        int64_t id_runs = 1;
        for (int64_t i = 1; i < n && id_runs <= PATCH_DMA_MAX_RUNS; ++i)
            if (blocks[i] != blocks[i - 1] + 1) ++id_runs;
        dma_patch = id_runs <= PATCH_DMA_MAX_RUNS;
    }
    const bool by_kernel = mode == PIE_MODE_KERNEL || mode == PIE_MODE_KERNEL_BULK;
    if (arrive != nullptr && ticket <= 0) arrive = nullptr;
    const bool need_list = by_kernel || slot_table_row != nullptr || arrive != nullptr;
    const int64_t body_len = ((dma_patch ? n : 3 * n) + 3) & ~int64_t(3);
    const int64_t list_len = body_len + (arrive ? 4 : 0);   // the ticket for the arrival word sits behind the list
    if (used_sm) *used_sm = by_kernel || (mode == PIE_MODE_COPY_ENGINE && slot_table_row != nullptr && !dma_patch);
    int64_t off = 0;
    if (need_list && dma_patch) {
        int st = list_alloc(p, list_len, &off);
        if (st != PIE_OK) return st;
        int32_t *h = p->list_host + off;
        for (int64_t i = 0; i < n; ++i) h[i] = dir_queue == PIE_Q_IN ? dst[i] : -1;
    } else if (need_list) {
        int st = list_alloc(p, list_len, &off);
        if (st != PIE_OK) return st;
        int32_t *h = p->list_host + off;
        for (int64_t i = 0; i < n && (by_kernel || slot_table_row != nullptr); ++i) {
            h[3 * i + 0] = src[i];
            h[3 * i + 1] = dst[i];
            h[3 * i + 2] = blocks ? blocks[i] : 0;
        }
        // the swap kernel wants its indices in device memory (no link latency per item); the table patch after
        // copy-engine copies reads the few entries straight from the pinned list and saves a copy-engine operation
        if (by_kernel)
            PIE_CUDA(cudaMemcpyAsync(p->list_dev + off, h, (size_t)(3 * n) * 4, cudaMemcpyHostToDevice, stream));
    }
    const int table_mode = slot_table_row ? (dir_queue == PIE_Q_IN ? 1 : 2) : 0;
    if (by_kernel) {
        const int ctas = p->cfg.swap_ctas > 0 ? p->cfg.swap_ctas : (mode == PIE_MODE_KERNEL ? 16 : 32);
        if (mode == PIE_MODE_KERNEL)
            PIE_CUDA(pie::launch_swap(src_pool, dst_pool, p->list_dev + off, n, BB, slot_table_row, table_mode, ctas, stream));
        else
            PIE_CUDA(pie::launch_swap_bulk(src_pool, dst_pool, p->list_dev + off, n, BB, slot_table_row, table_mode, ctas,
                                           p->status_dev, stream));
        p->stats.calls_kernel += 1;
    } else {
        // copy engine: one cudaMemcpyAsync per run of consecutive (src, dst) slots
        const cudaMemcpyKind kind = dir_queue == PIE_Q_IN ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
        int64_t i = 0;
        while (i < n) {
            if (elide && elide[i]) {
                ++i;
                continue;
            }
            int64_t j = i + 1;
            while (j < n && !(elide && elide[j]) && src[j] == src[j - 1] + 1 && dst[j] == dst[j - 1] + 1) ++j;
            PIE_CUDA(cudaMemcpyAsync(dst_pool + (int64_t)dst[i] * BB, src_pool + (int64_t)src[i] * BB, (size_t)((j - i) * BB),
                                     kind, stream));
            p->stats.copy_engine_copies += 1;
            i = j;
        }
        if (dma_patch) {
            const int32_t *h = p->list_host + off;
            for (int64_t a = 0; a < n;) {
                int64_t b = a + 1;
                while (b < n && blocks[b] == blocks[b - 1] + 1) ++b;
                PIE_CUDA(cudaMemcpyAsync(slot_table_row + blocks[a], h + a, (size_t)(b - a) * 4, cudaMemcpyHostToDevice, stream));
                a = b;
            }
        } else if (slot_table_row) {
            PIE_CUDA(pie::launch_patch_from_list(slot_table_row, p->list_host + off, n, table_mode, stream));
            p->stats.patch_kernel_launches += 1;
        }
        p->stats.calls_copy_engine += 1;
    }
    if (arrive) {
        unsigned long long *h = reinterpret_cast<unsigned long long *>(p->list_host + off + body_len);
        *h = (unsigned long long)ticket;
        PIE_CUDA(cudaMemcpyAsync(arrive, h, 8, cudaMemcpyHostToDevice, stream));
    }
    if (need_list) {
        if (ticket > 0) {
            list_commit_ticket(p, off, list_len, dir_queue, ticket);
        } else {
            int st = list_commit(p, off, list_len, stream);
            if (st != PIE_OK) return st;
        }
    }
    return PIE_OK;
}

int swap_prepare(pie_pool *p, int queue, int32_t layer, const int32_t *ids, int64_t n, SwapList *out) {
    out->layer = layer;
    out->ticket = out->n_moved = out->n_elided = 0;
    if (n == 0) return (layer < 0 || layer >= p->cfg.n_layers) ? PIE_ERR_RANGE : PIE_OK;
    out->moved.resize((size_t)n);
    out->src.resize((size_t)n);
    out->dst.resize((size_t)n);
    out->elide.resize((size_t)n);
    int st = p->table->swap(queue, layer, ids, n, &out->ticket, out->moved.data(), out->src.data(), out->dst.data(), &out->n_moved,
                            out->waits, out->elide.data());
    if (st != PIE_OK || out->n_moved == 0) return st;
    p->last_swap_step = p->step;
    for (int64_t i = 0; i < out->n_moved; ++i) out->n_elided += out->elide[(size_t)i];
    // a unit that is pushed out belongs to the host-resident set from now on; bringing it in for a layer's
    // turn does not take it out of the set (only a lower ratio does)
    if (queue == PIE_Q_OUT)
        for (int64_t i = 0; i < out->n_moved; ++i) {
            pie::Unit &u = p->table->unit(layer, out->moved[(size_t)i]);
            if (!u.home_host) {
                u.home_host = 1;
                p->home_count[(size_t)layer] += 1;
                p->home_dirty[(size_t)layer] = 1;
            }
        }
    return PIE_OK;
}

// Phase 1 is done: a failure from here on leaves the pool unusable (sticky) rather than inconsistent.
#define PIE_STICKY(expr)                  \
    do {                                  \
        int st__ = (expr);                \
        if (st__ != PIE_OK) {             \
            p->sticky = st__;             \
            return st__;                  \
        }                                 \
    } while (0)

void swap_account(pie_pool *p, int queue, const SwapList &l) {
    (queue == PIE_Q_IN ? p->stats.bytes_in : p->stats.bytes_out) += (double)(l.n_moved - l.n_elided) * (double)p->block_bytes;
    p->stats.bytes_out_elided += (double)l.n_elided * (double)p->block_bytes;
}

// not_before: a compute ticket the copy must not start before (0 = none).  The decode loop uses it to start a
// prefetch when the group of layers before it starts computing (Section 3.3), not as early as the host happens to run
// ahead: that keeps a unit on the host for as long as possible and the GPU staging share at a few layers' worth.
int swap_issue(pie_pool *p, int queue, SwapList &l, int32_t mode, int64_t not_before) {
    if (l.n_moved == 0) return PIE_OK;
    cudaStream_t stream = p->stream[queue];
    PIE_STICKY(reserve_ticket_event(p, queue, l.ticket));
    l.waits[PIE_Q_COMPUTE] = std::max(l.waits[PIE_Q_COMPUTE], not_before);
    for (int q = 1; q <= 3; ++q) PIE_STICKY(wait_ticket(p, stream, q, l.waits[q]));
    LayerEvents *le = timing_slot(p, l.layer);
    if (le && cudaEventRecord(queue == PIE_Q_IN ? le->in0 : le->out0, stream) != cudaSuccess) le = nullptr;
    bool used_sm = false;
    PIE_STICKY(do_copies(p, queue, l.src.data(), l.dst.data(), l.n_moved, l.moved.data(),
                         p->slot_table_dev + (int64_t)l.layer * p->cfg.n_logical_blocks, mode, stream, l.ticket, l.elide.data(),
                         queue == PIE_Q_IN ? p->arrive_dev + l.layer : nullptr, &used_sm));
    if (queue == PIE_Q_IN) {
        p->layer_in_last[(size_t)l.layer] = l.ticket;
        if (used_sm) p->layer_in_sm[(size_t)l.layer] = l.ticket;
    }
    PIE_STICKY(record_ticket(p, queue, l.ticket));
    if (le) {
        (queue == PIE_Q_IN ? le->in1 : le->out1) = p->ticket_ev[queue][l.ticket % EV_RING];
        (queue == PIE_Q_IN ? le->has_in : le->has_out) = true;
        p->lev_last[p->step % TIMING_RING][queue] = p->ticket_ev[queue][l.ticket % EV_RING];
    }
    swap_account(p, queue, l);
    return PIE_OK;
}

// The lists of a group of layers, issued together.  Where they can go by copy engine and every list moves one and the
// same run of block ids, the group costs the copy stream three operations instead of three per layer: the blocks of all
// lists in as few copies as their slots allow (slots handed out to consecutive requests are consecutive, so usually
// one), the table entries of all layers in one strided copy, the arrival words in one.  Every list's ticket completes
// when the group has.  Anything else goes list by list.
int swap_issue_group(pie_pool *p, int queue, std::vector<SwapList> &lists, int32_t mode, int64_t not_before) {
    std::vector<SwapList *> live;
    for (SwapList &l : lists)
        if (l.n_moved > 0) live.push_back(&l);
    if (live.empty()) return PIE_OK;
    const int32_t NB = p->cfg.n_logical_blocks;
    const int64_t BB = p->block_bytes;
    bool merge = live.size() > 1 && (mode == PIE_MODE_AUTO || mode == PIE_MODE_COPY_ENGINE);
    const int64_t n0 = live[0]->n_moved;
    for (size_t i = 0; merge && i < live.size(); ++i) {
        const SwapList &l = *live[i];
        merge = l.n_moved == n0 && l.layer == live[0]->layer + (int32_t)i && l.moved[0] == live[0]->moved[0];
        for (int64_t j = 1; merge && j < l.n_moved; ++j) merge = l.moved[(size_t)j] == l.moved[(size_t)j - 1] + 1;
    }
    // the copies of the whole group, coalesced across the lists
    struct Run {
        int64_t src, dst, len;
    };
    std::vector<Run> runs;
    if (merge) {
        for (SwapList *l : live)
            for (int64_t j = 0; j < l->n_moved; ++j) {
                if (l->elide[(size_t)j]) continue;
                const int64_t sj = l->src[(size_t)j], dj = l->dst[(size_t)j];
                if (!runs.empty() && runs.back().src + runs.back().len == sj && runs.back().dst + runs.back().len == dj) runs.back().len += 1;
                else runs.push_back({sj, dj, 1});
            }
        int64_t blocks = 0;
        for (const Run &r : runs) blocks += r.len;
        if (mode == PIE_MODE_AUTO && !runs.empty() &&
            !((blocks * BB) / (int64_t)runs.size() >= AUTO_COPY_ENGINE_RUN_BYTES || (int64_t)runs.size() <= AUTO_COPY_ENGINE_MAX_RUNS * (int64_t)live.size()))
            merge = false;   // scattered: the lists go through the gather/scatter kernel one by one
    }
    if (!merge) {
        for (SwapList *l : live) {
            int st = swap_issue(p, queue, *l, mode, not_before);
            if (st != PIE_OK) return st;
        }
        return PIE_OK;
    }
    cudaStream_t stream = p->stream[queue];
    int64_t waits[4] = {0, 0, 0, not_before};
    for (SwapList *l : live) {
        PIE_STICKY(reserve_ticket_event(p, queue, l->ticket));
        for (int q = 1; q <= 3; ++q) waits[q] = std::max(waits[q], l->waits[q]);
    }
    for (int q = 1; q <= 3; ++q) PIE_STICKY(wait_ticket(p, stream, q, waits[q]));
    // timing: the group's lists count as one, under its first layer
    LayerEvents *le = timing_slot(p, live[0]->layer);
    if (le && cudaEventRecord(queue == PIE_Q_IN ? le->in0 : le->out0, stream) != cudaSuccess) le = nullptr;
    const uint8_t *src_pool = queue == PIE_Q_IN ? p->host_base : p->gpu_base;
    uint8_t *dst_pool = queue == PIE_Q_IN ? p->gpu_base : p->host_base;
    const cudaMemcpyKind kind = queue == PIE_Q_IN ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToHost;
    for (const Run &r : runs)
        if (cudaMemcpyAsync(dst_pool + r.dst * BB, src_pool + r.src * BB, (size_t)(r.len * BB), kind, stream) != cudaSuccess) {
            p->sticky = PIE_ERR_CUDA;
            return PIE_ERR_CUDA;
        }
    // table entries: one row of n0 entries per layer in the pinned ring, one strided copy into the layers' rows;
    // arrival words (swap-in): the lists' tickets, one copy into the layers' consecutive words
    const int64_t k = (int64_t)live.size();
    const int64_t body = ((k * n0) + 3) & ~int64_t(3);
    const int64_t words = body + (queue == PIE_Q_IN ? ((2 * k + 3) & ~int64_t(3)) : 0);
    int64_t off = 0;
    PIE_STICKY(list_alloc(p, words, &off));
    int32_t *h = p->list_host + off;
    for (int64_t i = 0; i < k; ++i)
        for (int64_t j = 0; j < n0; ++j) h[i * n0 + j] = queue == PIE_Q_IN ? live[(size_t)i]->dst[(size_t)j] : -1;
    cudaError_t e = cudaMemcpy2DAsync(p->slot_table_dev + (int64_t)live[0]->layer * NB + live[0]->moved[0], (size_t)NB * 4, h, (size_t)n0 * 4,
                                      (size_t)n0 * 4, (size_t)k, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess && queue == PIE_Q_IN) {
        unsigned long long *t = reinterpret_cast<unsigned long long *>(h + body);
        for (int64_t i = 0; i < k; ++i) t[i] = (unsigned long long)live[(size_t)i]->ticket;
        e = cudaMemcpyAsync(p->arrive_dev + live[0]->layer, t, (size_t)k * 8, cudaMemcpyHostToDevice, stream);
    }
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        p->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    list_commit_ticket(p, off, words, queue, live.back()->ticket);
    p->stats.calls_copy_engine += (double)k;
    p->stats.copy_engine_copies += (double)runs.size();
    for (SwapList *l : live) {
        if (queue == PIE_Q_IN) p->layer_in_last[(size_t)l->layer] = l->ticket;
        PIE_STICKY(record_ticket(p, queue, l->ticket));
        swap_account(p, queue, *l);
    }
    if (le) {
        cudaEvent_t last = p->ticket_ev[queue][live.back()->ticket % EV_RING];
        (queue == PIE_Q_IN ? le->in1 : le->out1) = last;
        (queue == PIE_Q_IN ? le->has_in : le->has_out) = true;
        p->lev_last[p->step % TIMING_RING][queue] = last;
    }
    return PIE_OK;
}

int pool_swap(pie_pool *p, int queue, int32_t layer, const int32_t *ids, int64_t n, int32_t mode, int64_t not_before = 0) {
    if (!p) return PIE_ERR_INVALID;
    if (p->sticky != PIE_OK) return p->sticky;
    if (mode < PIE_MODE_AUTO || mode > PIE_MODE_KERNEL_BULK) return PIE_ERR_INVALID;
    if (n < 0 || (n > 0 && !ids)) return PIE_ERR_INVALID;
    int st = poll(p);
    if (st != PIE_OK) return st;
    SwapList &l = p->one_list;
    st = swap_prepare(p, queue, layer, ids, n, &l);
    if (st != PIE_OK) return st;
    return swap_issue(p, queue, l, mode, not_before);
}

// does the device take 64-bit stream memory operations (stream waits by value)?
bool can_wait_by_value(int dev) {
    void *f_get = nullptr, *f_attr = nullptr;
    cudaDriverEntryPointQueryResult q1, q2;
    if (cudaGetDriverEntryPoint("cuDeviceGet", &f_get, cudaEnableDefault, &q1) != cudaSuccess || q1 != cudaDriverEntryPointSuccess || !f_get)
        return false;
    if (cudaGetDriverEntryPoint("cuDeviceGetAttribute", &f_attr, cudaEnableDefault, &q2) != cudaSuccess ||
        q2 != cudaDriverEntryPointSuccess || !f_attr)
        return false;
    CUdevice cu_dev;
    if (reinterpret_cast<CUresult (*)(CUdevice *, int)>(f_get)(&cu_dev, dev) != CUDA_SUCCESS) return false;
    int can = 0;
    if (reinterpret_cast<CUresult (*)(int *, CUdevice_attribute, CUdevice)>(f_attr)(&can, CU_DEVICE_ATTRIBUTE_CAN_USE_64_BIT_STREAM_MEM_OPS,
                                                                                   cu_dev) != CUDA_SUCCESS)
        return false;
    return can != 0;
}

int sync_all(pie_pool *p, int64_t timeout_us) {
    const auto t0 = std::chrono::steady_clock::now();
    for (int q = 1; q <= 3; ++q) {
        for (;;) {
            cudaError_t e = cudaStreamQuery(p->stream[q]);
            if (e == cudaSuccess) break;
            if (e != cudaErrorNotReady) {
                g_last_cuda_error = (int)e;
                p->sticky = PIE_ERR_CUDA;
                return PIE_ERR_CUDA;
            }
            const auto us = std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now() - t0).count();
            if (timeout_us >= 0 && us > timeout_us) return PIE_ERR_TIMEOUT;
        }
    }
    // the compute stream is idle: every compute ticket enqueued so far has completed, marked or not
    p->compute_marks.clear();
    p->compute_marked = p->recorded[PIE_Q_COMPUTE];
    if (p->recorded[PIE_Q_COMPUTE] > p->table->done(PIE_Q_COMPUTE)) p->table->confirm(PIE_Q_COMPUTE, p->recorded[PIE_Q_COMPUTE]);
    return poll(p);
}

int patch_units(pie_pool *p, const std::vector<int32_t> &entries) {
    const int64_t n = (int64_t)entries.size() / 2;
    if (n == 0) return PIE_OK;
    // large updates go in pieces that fit the ring
    const int64_t piece = std::max<int64_t>(1, p->list_words / 8);
    for (int64_t done = 0; done < n; done += piece) {
        const int64_t m = std::min(piece, n - done);
        int64_t off;
        int st = list_alloc(p, 2 * m, &off);
        if (st != PIE_OK) return st;
        std::memcpy(p->list_host + off, entries.data() + 2 * done, (size_t)(2 * m) * 4);
        cudaStream_t s = p->stream[PIE_Q_COMPUTE];
        PIE_CUDA(cudaMemcpyAsync(p->list_dev + off, p->list_host + off, (size_t)(2 * m) * 4, cudaMemcpyHostToDevice, s));
        PIE_CUDA(pie::launch_patch(p->slot_table_dev, p->list_dev + off, m, s));
        st = list_commit(p, off, 2 * m, s);
        if (st != PIE_OK) return st;
    }
    return PIE_OK;
}

void destroy_pool(pie_pool *p) {
    if (!p) return;
    if (p->aux_stream) cudaStreamSynchronize(p->aux_stream);   // a stamp copy may still be writing the pinned buffer
    for (int q = 1; q <= 2; ++q)
        for (int i = 0; i < EV_RING; ++i)
            if (p->ticket_ev[q][i]) cudaEventDestroy(p->ticket_ev[q][i]);
    for (int i = 0; i < EV_RING; ++i) {
        if (p->compute_ev_plain[i]) cudaEventDestroy(p->compute_ev_plain[i]);
        if (p->compute_ev_stamped[i]) cudaEventDestroy(p->compute_ev_stamped[i]);
    }
    for (int i = 0; i < LIST_EVENTS; ++i)
        if (p->list_events[i]) cudaEventDestroy(p->list_events[i]);
    for (int k = 0; k < TIMING_RING; ++k)
        for (LayerEvents &e : p->lev[k])
            for (cudaEvent_t ev : {e.in0, e.out0})
                if (ev) cudaEventDestroy(ev);
    for (int k = 0; k < TIMING_RING; ++k) {
        if (p->lev_anchor[k]) cudaEventDestroy(p->lev_anchor[k]);
        if (p->lev_close_ev[k]) cudaEventDestroy(p->lev_close_ev[k]);
        if (p->step_end_ev[k]) cudaEventDestroy(p->step_end_ev[k]);
    }
    if (p->aux_stream) cudaStreamDestroy(p->aux_stream);
    for (int i = 0; i < 2; ++i)
        if (p->io_stream[i]) cudaStreamDestroy(p->io_stream[i]);
    if (p->own_streams)
        for (int q = 1; q <= 3; ++q)
            if (p->stream[q]) cudaStreamDestroy(p->stream[q]);
    if (p->own_gpu && p->gpu_base) cudaFree(p->gpu_base);
    if (p->own_host && p->host_base) cudaFreeHost(p->host_base);
    cudaFree(p->slot_table_dev);
    cudaFree(p->arrive_dev);
    cudaFree(p->io_arrive_dev);
    cudaFree(p->done_dev);
    cudaFree(p->list_dev);
    if (p->list_host) cudaFreeHost(p->list_host);
    if (p->status_host) cudaFreeHost(p->status_host);
    if (p->stamps_host) cudaFreeHost(p->stamps_host);
    cudaFree(p->stamps_dev);
    if (p->governor) pie_governor_destroy(p->governor);
    cudaFree(p->scratch.chunk_off);
    cudaFree(p->scratch.counters);
    cudaFree(p->scratch.part_o);
    cudaFree(p->scratch.part_ml);
    for (int t = 0; t < 2; ++t) {
        cudaFree(p->scratch.part_o_more[t]);
        cudaFree(p->scratch.part_ml_more[t]);
    }
    cudaFree(p->stage_q);
    cudaFree(p->stage_out);
    cudaFree(p->stage_k);
    cudaFree(p->stage_v);
    cudaFree(p->stage_bt);
    cudaFree(p->stage_ctx);
    delete p->fifo;
    delete p->table;
    delete p;
}

// A merge that was left to a next call that does not come (an error, a different batch): launch the combine kernel now.
int flush_deferred_combine(pie_pool *p) {
    if (!p->deferred.on) return PIE_OK;
    p->deferred.on = false;
    pie::AttnShape sh{p->cfg.head_dim, p->cfg.dtype, p->cfg.n_q_heads, p->cfg.n_kv_heads, p->cfg.n_logical_blocks,
                      p->cfg.n_gpu_slots, p->kv_fp8};
    cudaError_t e = pie::launch_combine(sh, p->scratch, p->deferred.out, p->deferred.n_seqs, p->deferred.max_blocks,
                                        p->deferred.split, p->deferred.parity, p->stream[PIE_Q_COMPUTE]);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        p->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    return PIE_OK;
}

// dependent: the call follows the previous layer's attention call of the same decode step directly, with the same
// lengths and tables: its kernel may be launched as a programmatic dependent of that call's last kernel.
// defer: the merge of this call's split-K partials is left to the next call's kernel (the caller promises that call, or
// flush_deferred_combine); a merge that an earlier call left (p->deferred) is taken on by this call's kernel.
int attention_call(pie_pool *p, int32_t layer, const void *q, void *out, const int32_t *bt_dev, int32_t max_blocks,
                   const int32_t *ctx_dev, const int32_t *bt_host, const int32_t *ctx_host, int32_t n_seqs, float scale,
                   const void *k_new, const void *v_new, bool dependent = false, bool defer = false, bool in_loop = false) {
    if (!p) return PIE_ERR_INVALID;
    if (p->sticky != PIE_OK) return p->sticky;
    if (layer < 0 || layer >= p->cfg.n_layers) return PIE_ERR_RANGE;
    if (!q || !out || !bt_dev || !ctx_dev || n_seqs < 0 || max_blocks <= 0) return PIE_ERR_INVALID;
    if (n_seqs > p->scratch.max_seqs) return PIE_ERR_INVALID;
    if ((k_new == nullptr) != (v_new == nullptr)) return PIE_ERR_INVALID;
    if ((bt_host == nullptr) != (ctx_host == nullptr)) return PIE_ERR_INVALID;
    int st = poll(p);
    if (st != PIE_OK) return st;
    st = check_status_word(p);  // a flag raised by an earlier call's kernels
    if (st != PIE_OK) return st;
    if (n_seqs == 0) return PIE_OK;
    // Split-K chunk.  In the decode loop consecutive layers' launches overlap at their ends, so a launch's slowest CTA no
    // longer holds the SMs up and long work items win (fewer partials, less work per token around the items): where the
    // caller left the choice to the library, the largest of 2048 / 1024 tokens that still gives every CTA an item (counted
    // from the blocks allocated) - measured on the three shapes: 6.27 -> 6.86, 6.60 -> 7.05 and 6.89 -> 7.22 TB/s against 512
    // / 1024 / 512 tokens.  Single calls keep the pool's chunk: nothing hides their tail.
    int64_t split = p->cfg.split_tokens;
    if (in_loop && p->auto_split) {
        const int64_t tokens = (int64_t)p->table->n_allocated() * 16;
        for (int64_t s = 2048; s > split; s /= 2)
            if (tokens / s * p->cfg.n_kv_heads >= p->attn_grid) {
                split = s;
                break;
            }
    }
    // host-side checks when the caller supplied host copies of the tables
    int64_t ticket = 0, waits[4];
    if (bt_host) {
        p->v_in.clear();
        int64_t chunks = 0;
        for (int32_t s = 0; s < n_seqs; ++s) {
            const int32_t ctx = ctx_host[s];
            if (ctx < 0 || ctx > max_blocks * 16) return PIE_ERR_INVALID;
            chunks += (ctx + split - 1) / split;
            for (int32_t b = 0; b < (ctx + 15) / 16; ++b) p->v_in.push_back(bt_host[(int64_t)s * max_blocks + b]);
        }
        if (chunks * p->cfg.n_kv_heads > p->scratch.max_items) return PIE_ERR_INVALID;
        st = p->table->attention(layer, p->v_in.data(), (int64_t)p->v_in.size(), &ticket, waits);
    } else {
        st = p->table->attention(layer, nullptr, 0, &ticket, waits);
    }
    if (st != PIE_OK) return st;
    if (k_new && p->table->tracks_writes()) {
        // kept host copies of the blocks this call's append writes go stale
        const int32_t NB = p->cfg.n_logical_blocks;
        auto mark = [&](int32_t b) {
            if (b >= 0 && b < NB && p->table->allocated(b)) p->table->unit(layer, b).dirty = 1;
        };
        if (bt_host) {
            for (int32_t s = 0; s < n_seqs; ++s)
                if (ctx_host[s] > 0) mark(bt_host[(int64_t)s * max_blocks + (ctx_host[s] - 1) / 16]);
        } else if (p->append_declared) {
            for (int32_t b : p->append_ids) mark(b);
        } else {
            p->table->mark_layer_dirty(layer);
        }
    }
    cudaStream_t stream = p->stream[PIE_Q_COMPUTE];
    st = reserve_ticket_event(p, PIE_Q_COMPUTE, ticket);
    if (st != PIE_OK) { p->sticky = st; return st; }
    LayerEvents *le = timing_slot(p, layer);
    // Presence wait (Section 3.2).  Units that a list of this layer is still bringing in: the kernel itself waits for the
    // layer's arrival word, so the compute stream carries no cross-stream wait (each costs the stream a few
    // microseconds, layer after layer).  Anything else - a list an SM kernel moves, a slot inherited from a copy of
    // another layer or direction - is waited for by the stream.
    unsigned long long arrive_need = 0;
    if (waits[PIE_Q_IN] > 0 && waits[PIE_Q_IN] <= p->layer_in_last[(size_t)layer] &&
        p->layer_in_sm[(size_t)layer] <= p->table->done(PIE_Q_IN)) {
        arrive_need = (unsigned long long)waits[PIE_Q_IN];
        waits[PIE_Q_IN] = 0;
    }
    for (int qd = 1; qd <= 2; ++qd) {
        if (le && waits[qd] > p->table->done(qd)) le->stream_wait = true;
        st = wait_ticket(p, stream, qd, waits[qd]);
        if (st != PIE_OK) { p->sticky = st; return st; }
    }
    pie::AttnShape sh{p->cfg.head_dim, p->cfg.dtype, p->cfg.n_q_heads, p->cfg.n_kv_heads, p->cfg.n_logical_blocks,
                      p->cfg.n_gpu_slots, p->kv_fp8};
    pie::AttnLaunch a{};
    a.k_scale = p->k_scale;
    a.v_scale = p->v_scale;
    a.q = q;
    a.out = out;
    a.block_table = bt_dev;
    a.max_blocks = max_blocks;
    a.ctx_lens = ctx_dev;
    a.slot_table = p->slot_table_dev + (int64_t)layer * p->cfg.n_logical_blocks;
    a.n_seqs = n_seqs;
    a.scale = scale;
    a.k_new = k_new;
    a.v_new = v_new;
    a.gpu_pool = p->gpu_base;
    a.split_tokens = (int32_t)split;
    a.grid = p->attn_grid;
    a.variant = p->cfg.attn_variant;
    a.status = p->status_dev;
    a.stamps = le ? stamp_dev(p, layer, STAMP_START) : nullptr;
    a.arrive = p->arrive_dev + layer;
    a.arrive_need = arrive_need;
    a.inputs_arrive = p->io_arrive_dev;
    a.inputs_need = p->inputs_need;
    a.done_word = p->done_dev;
    a.done_value = (unsigned long long)ticket;
    a.dependent_launch = dependent;
    // a merge the call before this one left: this kernel takes it on if it attends the same batch (else it is merged now)
    if (p->deferred.on && !(dependent && p->deferred.n_seqs == n_seqs && p->deferred.max_blocks == max_blocks && p->deferred.ctx == ctx_dev &&
                            p->deferred.split == (int32_t)split)) {
        st = flush_deferred_combine(p);
        if (st != PIE_OK) return st;
    }
    if (p->deferred.on) {
        a.prev_out = p->deferred.out;
        a.parity = (p->deferred.parity + 1) % 3;
    }
    a.defer_combine = defer;
    if (le && p->cfg.timing >= 2 && !p->lev_anchored[p->step % TIMING_RING]) {
        const int k = (int)(p->step % TIMING_RING);
        if (cudaEventRecord(p->lev_anchor[k], stream) == cudaSuccess) p->lev_anchored[k] = true;
    }
    cudaError_t e = pie::launch_attention(sh, p->scratch, a, p->use3d ? p->map3d : p->map2d, p->use3d, stream);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        p->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    p->deferred.on = defer && n_seqs > 0;
    p->deferred.out = out;
    p->deferred.parity = a.parity;
    p->deferred.n_seqs = n_seqs;
    p->deferred.max_blocks = max_blocks;
    p->deferred.ctx = ctx_dev;
    p->deferred.split = (int32_t)split;
    st = record_ticket(p, PIE_Q_COMPUTE, ticket);
    if (st != PIE_OK) p->sticky = st;
    p->last_attn_ticket = ticket;
    if (le && st == PIE_OK) {
        le->has_compute = true;
        p->lev_closed[p->step % TIMING_RING] = false;   // the set's newest compute ticket has no mark yet (close_step_set)
    }
    return st;
}

// The host enqueues at most two decode steps beyond the one the GPU is working on (pie_step_begin waits; one step of
// slack beyond the minimum, so that a few milliseconds' delay of the host thread does not leave the GPU idle).  Slots released by a step's swap lists can only be handed out as free for certain once their copies are
// known complete; a host that is several steps ahead finds nothing but slots still in flight, takes them in the order
// they were released, mixed with what has just come back, and the lists break into several runs (measured on 17 long
// sequences and 80 layers: 3 runs per list of 20 blocks, and the copy engines at 22 GB/s instead of 40).  The event is
// recorded on the side stream behind a wait by value for the step's last attention kernel: nothing on the compute stream.
int mark_step_end(pie_pool *p) {
    if (p->step <= 0 || !p->wait_value64 || !p->aux_stream || p->last_attn_ticket <= p->step_end_ticket) return PIE_OK;
    if (p->recorded[PIE_Q_COMPUTE] != p->last_attn_ticket) return PIE_OK;
    const int k = (int)(p->step % TIMING_RING);
    if (p->wait_value64((CUstream)p->aux_stream, (CUdeviceptr)(uintptr_t)p->done_dev, (cuuint64_t)p->last_attn_ticket,
                        CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) {
        g_last_cuda_error = (int)cudaErrorUnknown;
        return PIE_ERR_CUDA;
    }
    PIE_CUDA(cudaEventRecord(p->step_end_ev[k], p->aux_stream));
    p->step_end_of[k] = p->step;
    p->step_end_ticket = p->last_attn_ticket;
    return PIE_OK;
}

// The timing set of the step in progress is complete once its newest compute ticket is: give that ticket its mark.
int close_step_set(pie_pool *p) {
    if (!p->cfg.timing || p->step <= 0) return PIE_OK;
    const int k = (int)(p->step % TIMING_RING);
    if (p->lev_step[k] != p->step || p->lev_closed[k]) return PIE_OK;
    const size_t set_words = (size_t)p->cfg.n_layers * STAMP_WORDS;
    if (p->wait_value64 && p->aux_stream && p->recorded[PIE_Q_COMPUTE] == p->last_attn_ticket) {
        // a side stream waits for the step's last attention kernel by value, copies the stamps and records the event
        // that closes the set: the compute stream carries nothing between two steps
        if (p->wait_value64((CUstream)p->aux_stream, (CUdeviceptr)(uintptr_t)p->done_dev, (cuuint64_t)p->last_attn_ticket,
                            CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS) {
            g_last_cuda_error = (int)cudaErrorUnknown;
            return PIE_ERR_CUDA;
        }
        PIE_CUDA(cudaMemcpyAsync(p->stamps_host + (size_t)k * set_words, p->stamps_dev + (size_t)k * set_words, set_words * 8,
                                 cudaMemcpyDeviceToHost, p->aux_stream));
        PIE_CUDA(cudaEventRecord(p->lev_close_ev[k], p->aux_stream));
        p->lev_last[k][PIE_Q_COMPUTE] = p->lev_close_ev[k];
        p->lev_closed[k] = true;
        return PIE_OK;
    }
    PIE_CUDA(cudaMemcpyAsync(p->stamps_host + (size_t)k * set_words, p->stamps_dev + (size_t)k * set_words, set_words * 8,
                             cudaMemcpyDeviceToHost, p->stream[PIE_Q_COMPUTE]));
    cudaEvent_t ev = nullptr;
    int st = push_mark(p, &ev);   // behind the copy
    if (st != PIE_OK) return st;
    p->lev_last[k][PIE_Q_COMPUTE] = ev;
    p->lev_closed[k] = true;
    return PIE_OK;
}

// the host-resident set of `layer` follows the ratio: mark / unmark units in id order
// The GPU pool must hold every layer's resident share plus the host shares in transit (the layer computing and the
// layers being prefetched): L (n - h) + transit * h <= n_gpu_slots bounds the host-resident count h of a layer
// from below.
int64_t min_home_count(const pie_pool *p) {
    const int64_t n_alloc = p->table->n_allocated(), L = p->cfg.n_layers;
    // the group that computes + the group being prefetched; a group is one layer unless the caller asked for more
    const int64_t transit = std::min<int64_t>(2 * std::max(1, p->group_setting), L);
    if (L <= transit) return 0;
    const int64_t deficit = L * n_alloc - p->cfg.n_gpu_slots;
    return deficit > 0 ? std::min(n_alloc, (deficit + L - transit - 1) / (L - transit)) : 0;
}

// the smallest extension ratio the GPU pool's size allows with the blocks allocated now
double ratio_floor(const pie_pool *p) {
    const int64_t n_alloc = p->table->n_allocated();
    return n_alloc > 0 ? (double)min_home_count(p) / (double)n_alloc : 0.0;
}

void apply_ratio_to_layer(pie_pool *p, int32_t layer) {
    if (p->ratio_mode == 0) return;
    const int32_t NB = p->cfg.n_logical_blocks;
    const int64_t n_alloc = p->table->n_allocated();
    const int64_t target = std::max((int64_t)std::llround(p->ratio * (double)n_alloc), min_home_count(p));
    int64_t &count = p->home_count[(size_t)layer];
    if (count != target) p->home_dirty[(size_t)layer] = 1;
    if (count < target) {
        for (int32_t b = 0; b < NB && count < target; ++b) {
            if (!p->table->allocated(b)) continue;
            pie::Unit &u = p->table->unit(layer, b);
            if (!u.home_host) { u.home_host = 1; ++count; }
        }
    } else if (count > target) {
        for (int32_t b = NB - 1; b >= 0 && count > target; --b) {
            if (!p->table->allocated(b)) continue;
            pie::Unit &u = p->table->unit(layer, b);
            if (u.home_host) {
                u.home_host = 0;
                --count;
                p->table->drop_host_copy(layer, b);  // a kept host slot is only for members of the set
            }
        }
    }
}

// The units of `layer` that a plan has to look at, in ascending id: members of the host-resident set and units
// that are on the host for any other reason.  Rebuilt by one scan only after the set changed (an allocation, a
// free, a ratio change, a caller's own swap-out), so that a steady decode loop does not walk every block of
// every layer on every step.
const std::vector<int32_t> &candidate_ids(pie_pool *p, int32_t layer) {
    std::vector<int32_t> &v = p->home_list[(size_t)layer];
    if (p->home_dirty[(size_t)layer]) {
        v.clear();
        const int32_t NB = p->cfg.n_logical_blocks;
        for (int32_t b = 0; b < NB; ++b) {
            if (!p->table->allocated(b)) continue;
            const pie::Unit &u = p->table->unit(layer, b);
            if (u.home_host || u.side == PIE_HOST) v.push_back(b);
        }
        p->home_dirty[(size_t)layer] = 0;
    }
    return v;
}

// the units of `target` that are still on the host, as many as the GPU pool can take: hottest first (Section 3.3)
int plan_in(pie_pool *p, int32_t target, std::vector<int32_t> &in_ids) {
    in_ids.clear();
    apply_ratio_to_layer(p, target);
    int64_t room = p->table->gpu_available();
    int64_t left_behind = 0;
    for (int32_t b : candidate_ids(p, target)) {
        const pie::Unit &u = p->table->unit(target, b);
        if (u.side == PIE_HOST) {
            if (room > 0) {
                in_ids.push_back(b);
                --room;
            } else {
                ++left_behind;
            }
        } else if (!u.home_host) {
            p->home_dirty[(size_t)target] = 1;  // left the set and is back on the GPU: drop it at the next rebuild
            p->table->drop_host_copy(target, b);
        }
    }
    return left_behind == 0 ? PIE_OK : PIE_ERR_NOMEM;
}

// coldest: this layer's host-home units go back once it has computed
void plan_out(pie_pool *p, int32_t layer, std::vector<int32_t> &out_ids) {
    out_ids.clear();
    p->table->layer_pass(layer);  // a resize in progress takes effect once every layer has been here (Section 4.1)
    apply_ratio_to_layer(p, layer);
    for (int32_t b : candidate_ids(p, layer)) {
        const pie::Unit &u = p->table->unit(layer, b);
        if (u.home_host && u.side == PIE_GPU) out_ids.push_back(b);
    }
}

int plan_layer(pie_pool *p, int32_t layer, std::vector<int32_t> &in_ids, std::vector<int32_t> &out_ids) {
    plan_out(p, layer, out_ids);
    return plan_in(p, (layer + 1) % p->cfg.n_layers, in_ids);
}

// How many consecutive layers the decode loop treats as one group (their prefetches are issued together when the
// group before them starts, their write-backs together when they have all computed: one mark on the compute stream
// per group instead of one per layer).  A group in use, the next one arriving and the previous one leaving occupy GPU
// slots at the same time, so the size follows what the pool can spare: three groups' host-resident shares.
int32_t group_layers(pie_pool *p) {
    const int32_t L = p->cfg.n_layers;
    if (p->group_setting > 0) return std::max(1, std::min(p->group_setting, L / 2));
    const int32_t cap = std::max(1, std::min(MAX_GROUP_LAYERS, L / 4));
    const int64_t n_alloc = p->table->n_allocated();
    int64_t h = p->ratio_mode != 0 ? std::max((int64_t)std::llround(p->ratio * (double)n_alloc), min_home_count(p)) : 0;
    int64_t resident = 0;
    for (int32_t l = 0; l < L; ++l) {
        h = std::max(h, p->home_count[(size_t)l]);
        resident += n_alloc - p->home_count[(size_t)l];
    }
    if (h <= 0) return cap;
    const int64_t spare = p->cfg.n_gpu_slots - std::max<int64_t>(resident, (int64_t)L * (n_alloc - h));
    return (int32_t)std::max<int64_t>(1, std::min<int64_t>(cap, spare / (3 * h)));
}

// The layers of the group in progress that have computed push their host-resident shares out (Section 3.3: the layer
// that has just finished is the coldest); the group is closed.
int finish_group(pie_pool *p) {
    if (p->group_done.empty()) {
        p->group_len = 0;
        return PIE_OK;
    }
    if (p->sticky != PIE_OK) return p->sticky;
    struct PollHold {
        pie_pool *p;
        bool was;
        ~PollHold() { p->poll_hold = was; }
    } hold{p, p->poll_hold};
    p->poll_hold = true;
    std::vector<int32_t> layers;
    layers.swap(p->group_done);
    p->group_len = 0;
    if (p->group_lists.size() < layers.size()) p->group_lists.resize(layers.size());
    std::vector<SwapList> &lists = p->group_lists;
    for (SwapList &l : lists) l.n_moved = 0;
    int st = PIE_OK;
    size_t n_lists = 0;
    for (int32_t l : layers) {
        plan_out(p, l, p->v_plan_out);
        if (p->cfg.n_layers <= 1 || p->v_plan_out.empty()) continue;
        st = swap_prepare(p, PIE_Q_OUT, l, p->v_plan_out.data(), (int64_t)p->v_plan_out.size(), &lists[n_lists++]);
        if (st != PIE_OK) break;   // what was prepared before it still has to be issued
    }
    const int st2 = swap_issue_group(p, PIE_Q_OUT, lists, p->group_mode, 0);
    return st != PIE_OK ? st : st2;
}

// streams and the arrival word of the host-buffer entry point's pipeline (created at its first use)
int ensure_io(pie_pool *p) {
    if (p->io_stream[0]) return PIE_OK;
    PIE_CUDA(cudaStreamCreateWithFlags(&p->io_stream[0], cudaStreamNonBlocking));
    PIE_CUDA(cudaStreamCreateWithFlags(&p->io_stream[1], cudaStreamNonBlocking));
    PIE_CUDA(cudaMalloc((void **)&p->io_arrive_dev, 64));
    PIE_CUDA(cudaMemset(p->io_arrive_dev, 0, 64));
    return PIE_OK;
}

int ensure_stage(pie_pool *p, int32_t n_seqs, int32_t max_blocks) {
    const int64_t E = 2;
    const int64_t qb = (int64_t)p->cfg.n_layers * n_seqs * p->cfg.n_q_heads * p->cfg.head_dim * E;
    const int64_t kb = (int64_t)p->cfg.n_layers * n_seqs * p->cfg.n_kv_heads * p->cfg.head_dim * E;
    if (qb > p->stage_q_bytes) {
        cudaFree(p->stage_q);
        cudaFree(p->stage_out);
        p->stage_q = p->stage_out = nullptr;
        p->stage_q_bytes = 0;
        PIE_CUDA(cudaMalloc(&p->stage_q, (size_t)qb));
        PIE_CUDA(cudaMalloc(&p->stage_out, (size_t)qb));
        p->stage_q_bytes = qb;
    }
    if (kb > p->stage_kv_bytes) {
        cudaFree(p->stage_k);
        cudaFree(p->stage_v);
        p->stage_k = p->stage_v = nullptr;
        p->stage_kv_bytes = 0;
        PIE_CUDA(cudaMalloc(&p->stage_k, (size_t)kb));
        PIE_CUDA(cudaMalloc(&p->stage_v, (size_t)kb));
        p->stage_kv_bytes = kb;
    }
    const int64_t bw = (int64_t)n_seqs * max_blocks;
    if (bw > p->stage_bt_words) {
        cudaFree(p->stage_bt);
        p->stage_bt = nullptr;
        p->stage_bt_words = 0;
        PIE_CUDA(cudaMalloc(&p->stage_bt, (size_t)bw * 4));
        p->stage_bt_words = bw;
    }
    if (!p->stage_ctx) PIE_CUDA(cudaMalloc(&p->stage_ctx, (size_t)p->scratch.max_seqs * 4));
    return PIE_OK;
}

}  // namespace

// =========================================================================================================
// C ABI
// =========================================================================================================
extern "C" {

const char *pie_status_str(int status) {
    switch (status) {
        case PIE_OK: return "ok";
        case PIE_ERR_INVALID: return "invalid argument";
        case PIE_ERR_RANGE: return "id out of range";
        case PIE_ERR_NOMEM: return "no free slot / out of memory";
        case PIE_ERR_BUSY: return "unit busy (copy in flight)";
        case PIE_ERR_NOT_RESIDENT: return "unit not resident on the GPU";
        case PIE_ERR_TIMEOUT: return "timeout";
        case PIE_ERR_CUDA: return "CUDA error";
        case PIE_ERR_UNSUPPORTED: return "unsupported configuration";
        default: return "unknown status";
    }
}

int pie_last_cuda_error(void) { return g_last_cuda_error; }

size_t pie_block_bytes(const pie_pool *pool) { return pool ? (size_t)pool->block_bytes : 0; }

int pie_pool_create(const pie_pool_config *cfg_in, pie_pool **out) {
    if (!cfg_in || !out) return PIE_ERR_INVALID;
    // the caller's struct may be older (shorter) or newer (longer) than this build's: take what both know
    if (cfg_in->struct_size < offsetof(pie_pool_config, timing) + sizeof(int32_t)) return PIE_ERR_INVALID;
    pie_pool_config cfg_local;
    std::memset(&cfg_local, 0, sizeof cfg_local);
    std::memcpy(&cfg_local, cfg_in, std::min<size_t>(cfg_in->struct_size, sizeof cfg_local));
    cfg_local.struct_size = (uint32_t)sizeof cfg_local;
    const pie_pool_config *cfg = &cfg_local;
    if (cfg->n_layers <= 0 || cfg->n_q_heads <= 0 || cfg->n_kv_heads <= 0 || cfg->n_logical_blocks <= 0 ||
        cfg->n_gpu_slots <= 0 || cfg->n_host_slots < 0 || cfg->max_seqs <= 0)
        return PIE_ERR_INVALID;
    if (cfg->n_q_heads % cfg->n_kv_heads != 0) return PIE_ERR_INVALID;
    if (cfg->dtype != PIE_F16 && cfg->dtype != PIE_BF16) return PIE_ERR_INVALID;
    if (cfg->block_tokens != 16 || (cfg->head_dim != 64 && cfg->head_dim != 128)) return PIE_ERR_UNSUPPORTED;
    if (cfg->n_q_heads / cfg->n_kv_heads > 8) return PIE_ERR_UNSUPPORTED;
    if (cfg->kv_format != 0 && cfg->kv_format != 1) return PIE_ERR_INVALID;
    if (cfg->kv_format == 1 && (cfg->head_dim != 128 || cfg->attn_variant < 0 || cfg->attn_variant > 2)) return PIE_ERR_UNSUPPORTED;
    if (cfg->split_tokens < 0 || cfg->split_tokens % 16 != 0) return PIE_ERR_INVALID;
    if (cfg->gpu_base && ((uintptr_t)cfg->gpu_base & 127)) return PIE_ERR_INVALID;
    if ((uint64_t)cfg->n_gpu_slots * (uint64_t)cfg->n_kv_heads * 32u > 0x7fffffffull) return PIE_ERR_UNSUPPORTED;

    int n_dev = 0;
    PIE_CUDA(cudaGetDeviceCount(&n_dev));
    if (n_dev <= 0) {
        g_last_cuda_error = (int)cudaErrorNoDevice;
        return PIE_ERR_CUDA;
    }
    int dev = 0;
    PIE_CUDA(cudaGetDevice(&dev));
    cudaDeviceProp prop;
    PIE_CUDA(cudaGetDeviceProperties(&prop, dev));
    if (prop.major < 10) return PIE_ERR_UNSUPPORTED;  // built for sm_100a only

    pie_pool *p = new (std::nothrow) pie_pool();
    if (!p) return PIE_ERR_NOMEM;
    p->cfg = *cfg;
    // Split-K chunk: 512 tokens balances the persistent grid best on batches of many short sequences; where the pool
    // is laid out for few long ones (>= 6144 tokens per sequence on average) 1024 halves the partials and the merge
    // (measured: +6.5 % on 17 sequences of 4k-32k tokens with 8-head groups, -1.5 % on the batched shapes).
    p->auto_split = p->cfg.split_tokens == 0;
    if (p->cfg.split_tokens == 0)
        p->cfg.split_tokens = (int64_t)cfg->n_logical_blocks * 16 / std::max(cfg->max_seqs, 1) >= 6144 ? 1024 : 512;
    p->kv_fp8 = cfg->kv_format;
    p->block_bytes = (int64_t)2 * 16 * cfg->n_kv_heads * cfg->head_dim * (p->kv_fp8 ? 1 : 2);
    p->n_sms = prop.multiProcessorCount;
    p->table = new (std::nothrow) pie::Table(cfg->n_layers, cfg->n_logical_blocks, cfg->n_gpu_slots, cfg->n_host_slots);
    if (!p->table) { destroy_pool(p); return PIE_ERR_NOMEM; }
    if (cfg->visible_blocks != 0 && p->table->init_capacity(cfg->visible_blocks) != PIE_OK) { destroy_pool(p); return PIE_ERR_INVALID; }
    p->home_count.assign((size_t)cfg->n_layers, 0);
    p->home_list.assign((size_t)cfg->n_layers, std::vector<int32_t>());
    p->home_dirty.assign((size_t)cfg->n_layers, 1);

#define PIE_TRY(call, code)                            \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) {                      \
            g_last_cuda_error = (int)e__;              \
            destroy_pool(p);                           \
            return (code);                             \
        }                                              \
    } while (0)

    if (cfg->gpu_base) p->gpu_base = (uint8_t *)cfg->gpu_base;
    else {
        PIE_TRY(cudaMalloc((void **)&p->gpu_base, (size_t)(cfg->n_gpu_slots * p->block_bytes)), PIE_ERR_NOMEM);
        p->own_gpu = true;
    }
    if (cfg->host_base) p->host_base = (uint8_t *)cfg->host_base;
    else if (cfg->n_host_slots > 0) {
        PIE_TRY(cudaHostAlloc((void **)&p->host_base, (size_t)(cfg->n_host_slots * p->block_bytes), cudaHostAllocDefault),
                PIE_ERR_NOMEM);
        p->own_host = true;
    }
    if (cfg->own_streams) {
        int lo = 0, hi = 0;
        PIE_TRY(cudaDeviceGetStreamPriorityRange(&lo, &hi), PIE_ERR_CUDA);
        PIE_TRY(cudaStreamCreateWithPriority(&p->stream[PIE_Q_COMPUTE], cudaStreamNonBlocking, lo), PIE_ERR_CUDA);
        PIE_TRY(cudaStreamCreateWithPriority(&p->stream[PIE_Q_IN], cudaStreamNonBlocking, hi), PIE_ERR_CUDA);
        PIE_TRY(cudaStreamCreateWithPriority(&p->stream[PIE_Q_OUT], cudaStreamNonBlocking, hi), PIE_ERR_CUDA);
        p->own_streams = true;
    } else {
        p->stream[PIE_Q_COMPUTE] = (cudaStream_t)cfg->compute_stream;
        p->stream[PIE_Q_IN] = (cudaStream_t)cfg->copy_in_stream;
        p->stream[PIE_Q_OUT] = (cudaStream_t)cfg->copy_out_stream;
    }
    for (int q = 1; q <= 2; ++q)
        for (int i = 0; i < EV_RING; ++i)  // with timing on, a copy ticket's event doubles as the "end" mark of its list
            PIE_TRY(cudaEventCreateWithFlags(&p->ticket_ev[q][i], cfg->timing ? cudaEventDefault : cudaEventDisableTiming), PIE_ERR_CUDA);
    for (int i = 0; i < EV_RING; ++i) {
        PIE_TRY(cudaEventCreateWithFlags(&p->compute_ev_plain[i], cudaEventDisableTiming), PIE_ERR_CUDA);
        PIE_TRY(cudaEventCreateWithFlags(&p->compute_ev_stamped[i], cudaEventDefault), PIE_ERR_CUDA);
        p->ticket_ev[PIE_Q_COMPUTE][i] = p->compute_ev_plain[i];
    }
    for (int i = 0; i < LIST_EVENTS; ++i) PIE_TRY(cudaEventCreateWithFlags(&p->list_events[i], cudaEventDisableTiming), PIE_ERR_CUDA);
    PIE_TRY(cudaStreamCreateWithFlags(&p->aux_stream, cudaStreamNonBlocking), PIE_ERR_CUDA);
    for (int k = 0; k < TIMING_RING; ++k) PIE_TRY(cudaEventCreateWithFlags(&p->step_end_ev[k], cudaEventDisableTiming), PIE_ERR_CUDA);
    if (cfg->timing) {
        for (int k = 0; k < TIMING_RING; ++k) {
            p->lev[k].resize((size_t)cfg->n_layers);
            for (LayerEvents &e : p->lev[k])
                for (cudaEvent_t *ev : {&e.in0, &e.out0})
                    PIE_TRY(cudaEventCreate(ev), PIE_ERR_CUDA);
        }
        if (cfg->timing >= 2)
            for (int k = 0; k < TIMING_RING; ++k) PIE_TRY(cudaEventCreate(&p->lev_anchor[k]), PIE_ERR_CUDA);
        for (int k = 0; k < TIMING_RING; ++k) PIE_TRY(cudaEventCreateWithFlags(&p->lev_close_ev[k], cudaEventDisableTiming), PIE_ERR_CUDA);
        // The kernels note their stamps in device memory and one copy per step brings a step's set to the host.  (Stamps
        // in host-visible memory made every kernel end with a store across the host link; while swap lists were being
        // copied out that store queued behind them, and the next kernel started 30 us late, layer after layer.)
        const size_t stamp_bytes = (size_t)TIMING_RING * (size_t)cfg->n_layers * STAMP_WORDS * 8;
        PIE_TRY(cudaHostAlloc((void **)&p->stamps_host, stamp_bytes, cudaHostAllocDefault), PIE_ERR_NOMEM);
        std::memset(p->stamps_host, 0, stamp_bytes);
        PIE_TRY(cudaMalloc((void **)&p->stamps_dev, stamp_bytes), PIE_ERR_NOMEM);
        PIE_TRY(cudaMemset(p->stamps_dev, 0, stamp_bytes), PIE_ERR_CUDA);
    }
    const size_t table_bytes = (size_t)cfg->n_layers * (size_t)cfg->n_logical_blocks * 4;
    PIE_TRY(cudaMalloc((void **)&p->slot_table_dev, table_bytes), PIE_ERR_NOMEM);
    PIE_TRY(cudaMemset(p->slot_table_dev, 0xff, table_bytes), PIE_ERR_CUDA);
    PIE_TRY(cudaMalloc((void **)&p->done_dev, 64), PIE_ERR_NOMEM);
    PIE_TRY(cudaMemset(p->done_dev, 0, 64), PIE_ERR_CUDA);
    {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuStreamWaitValue64", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess && fn != nullptr) {
            if (can_wait_by_value(dev)) p->wait_value64 = reinterpret_cast<decltype(p->wait_value64)>(fn);
        }
    }
    PIE_TRY(cudaMalloc((void **)&p->arrive_dev, (size_t)cfg->n_layers * 8), PIE_ERR_NOMEM);
    PIE_TRY(cudaMemset(p->arrive_dev, 0, (size_t)cfg->n_layers * 8), PIE_ERR_CUDA);
    p->layer_in_sm.assign((size_t)cfg->n_layers, 0);
    p->layer_in_last.assign((size_t)cfg->n_layers, 0);
    p->list_words = std::max<int64_t>(1 << 20, (int64_t)cfg->n_logical_blocks * 3 * 8);
    PIE_TRY(cudaHostAlloc((void **)&p->list_host, (size_t)p->list_words * 4, cudaHostAllocDefault), PIE_ERR_NOMEM);
    PIE_TRY(cudaMalloc((void **)&p->list_dev, (size_t)p->list_words * 4), PIE_ERR_NOMEM);
    PIE_TRY(cudaHostAlloc((void **)&p->status_host, 64, cudaHostAllocMapped), PIE_ERR_NOMEM);
    std::memset(p->status_host, 0, 64);
    PIE_TRY(cudaHostGetDevicePointer((void **)&p->status_dev, p->status_host, 0), PIE_ERR_CUDA);

    // attention scratch: every chunk of every sequence, all KV heads
    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    const int64_t max_chunks = ((int64_t)cfg->n_logical_blocks * 16 + p->cfg.split_tokens - 1) / p->cfg.split_tokens + cfg->max_seqs;
    p->scratch.max_items = max_chunks * cfg->n_kv_heads;
    p->scratch.max_seqs = cfg->max_seqs;
    PIE_TRY(cudaMalloc((void **)&p->scratch.chunk_off, (size_t)(cfg->max_seqs + 1) * 4), PIE_ERR_NOMEM);
    {
        const size_t words = (size_t)pie::attn_counter_words(cfg->max_seqs, cfg->n_kv_heads);
        PIE_TRY(cudaMalloc((void **)&p->scratch.counters, words * 4), PIE_ERR_NOMEM);
        PIE_TRY(cudaMemset(p->scratch.counters, 0, words * 4), PIE_ERR_CUDA);  // the kernel leaves them at zero again
    }
    PIE_TRY(cudaMalloc((void **)&p->scratch.part_o, (size_t)(p->scratch.max_items * G * cfg->head_dim) * 4), PIE_ERR_NOMEM);
    PIE_TRY(cudaMalloc((void **)&p->scratch.part_ml, (size_t)(p->scratch.max_items * G * 2) * 4), PIE_ERR_NOMEM);
    // two more pairs: the decode step defers every layer's merge into the next layer's kernel, which starts beside this
    // layer's tail (three launches' buffers and counters are in use at a time at most)
    for (int t = 0; t < 2; ++t) {
        PIE_TRY(cudaMalloc((void **)&p->scratch.part_o_more[t], (size_t)(p->scratch.max_items * G * cfg->head_dim) * 4), PIE_ERR_NOMEM);
        PIE_TRY(cudaMalloc((void **)&p->scratch.part_ml_more[t], (size_t)(p->scratch.max_items * G * 2) * 4), PIE_ERR_NOMEM);
    }
    if (p->kv_fp8) {
        PIE_TRY(pie::make_pool_tensor_map_fp8(p->gpu_base, cfg->n_gpu_slots, cfg->n_kv_heads, &p->map2d), PIE_ERR_CUDA);
        p->use3d = 0;
    } else {
        PIE_TRY(pie::make_pool_tensor_maps(p->gpu_base, cfg->n_gpu_slots, cfg->n_kv_heads, cfg->head_dim, &p->map3d, &p->map2d,
                                           &p->use3d),
                PIE_ERR_CUDA);
        if (const char *env = std::getenv("PIE_TMA_2D"))
            if (env[0] == '1') p->use3d = 0;
        PIE_TRY(pie::make_prefill_tensor_map(p->gpu_base, cfg->n_gpu_slots, cfg->n_kv_heads, cfg->head_dim, &p->map_prefill), PIE_ERR_CUDA);
    }
    int per_sm = 0;
    PIE_TRY(pie::attn_configure(cfg->head_dim, cfg->dtype, cfg->attn_variant, &per_sm, p->kv_fp8), PIE_ERR_CUDA);
    if (per_sm <= 0) { destroy_pool(p); return PIE_ERR_UNSUPPORTED; }
    if (cfg->attn_ctas_per_sm > 0) per_sm = std::min(per_sm, cfg->attn_ctas_per_sm);
    p->attn_grid = per_sm * p->n_sms;
#undef PIE_TRY
    *out = p;
    return PIE_OK;
}

int pie_pool_destroy(pie_pool *pool) {
    if (!pool) return PIE_OK;
    int st = sync_all(pool, 10 * 1000 * 1000);
    destroy_pool(pool);
    return st == PIE_ERR_TIMEOUT ? st : PIE_OK;
}

int pie_block_alloc(pie_pool *pool, int64_t n, const uint8_t *on_host, int32_t *ids_out) {
    if (!pool || n < 0 || (n > 0 && !ids_out)) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    pie::Table *t = pool->table;
    const int32_t NB = pool->cfg.n_logical_blocks, L = pool->cfg.n_layers;
    // ids: the lowest free ones below the size visible now (a resize in progress: Section 4.1); slots are
    // handed out layer by layer (consecutive slots within a layer)
    const int32_t limit = t->alloc_limit();
    int32_t next = 0;
    for (int64_t i = 0; i < n; ++i) {
        while (next < limit && t->allocated(next)) ++next;
        if (next >= limit) return PIE_ERR_NOMEM;
        ids_out[i] = next++;
    }
    st = t->alloc_bulk(ids_out, n, on_host);
    if (st != PIE_OK) return st;  // all or nothing: the table is unchanged
    std::fill(pool->home_dirty.begin(), pool->home_dirty.end(), (uint8_t)1);
    std::vector<int32_t> entries;
    entries.reserve((size_t)(n * L * 2));
    for (int64_t i = 0; i < n; ++i)
        for (int32_t l = 0; l < L; ++l) {
            const pie::Unit &u = t->unit(l, ids_out[i]);
            if (u.home_host) pool->home_count[(size_t)l] += 1;
            if (u.side == PIE_GPU) {
                entries.push_back(l * NB + ids_out[i]);
                entries.push_back(u.gpu_slot);
            }
        }
    st = patch_units(pool, entries);
    if (st != PIE_OK) pool->sticky = st;
    return st;
}

int pie_block_free(pie_pool *pool, const int32_t *ids, int64_t n) {
    if (!pool || n < 0 || (n > 0 && !ids)) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    pie::Table *t = pool->table;
    const int32_t NB = pool->cfg.n_logical_blocks, L = pool->cfg.n_layers;
    for (int64_t i = 0; i < n; ++i) {
        if (ids[i] < 0 || ids[i] >= NB) return PIE_ERR_RANGE;
        if (!t->allocated(ids[i])) return PIE_ERR_INVALID;
        for (int64_t j = 0; j < i; ++j)
            if (ids[j] == ids[i]) return PIE_ERR_INVALID;
        for (int32_t l = 0; l < L; ++l)
            if (t->in_flight(t->unit(l, ids[i]))) return PIE_ERR_BUSY;
    }
    std::vector<int32_t> entries;
    std::fill(pool->home_dirty.begin(), pool->home_dirty.end(), (uint8_t)1);
    for (int64_t i = 0; i < n; ++i) {
        for (int32_t l = 0; l < L; ++l) {
            const pie::Unit &u = t->unit(l, ids[i]);
            if (u.home_host) pool->home_count[(size_t)l] -= 1;
            if (u.side == PIE_GPU) {
                entries.push_back(l * NB + ids[i]);
                entries.push_back(-1);
            }
        }
        t->free_block(ids[i]);
    }
    st = patch_units(pool, entries);
    if (st != PIE_OK) pool->sticky = st;
    return st;
}

static int unit_access(pie_pool *pool, int32_t layer, int32_t block, void *host_buf, bool write) {
    if (!pool || !host_buf) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (layer < 0 || layer >= pool->cfg.n_layers || block < 0 || block >= pool->cfg.n_logical_blocks) return PIE_ERR_RANGE;
    if (!pool->table->allocated(block)) return PIE_ERR_INVALID;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    pie::Unit &u = pool->table->unit(layer, block);
    if (pool->table->in_flight(u) || write) {
        // wait for the copies on the unit; a write must also not race an attention call still reading it
        st = sync_all(pool, 30 * 1000 * 1000);
        if (st != PIE_OK) return st;
    }
    uint8_t *p = u.side == PIE_GPU ? pool->gpu_base + (int64_t)u.gpu_slot * pool->block_bytes
                                   : pool->host_base + (int64_t)u.host_slot * pool->block_bytes;
    if (u.side == PIE_GPU) {
        if (write) PIE_CUDA(cudaMemcpy(p, host_buf, (size_t)pool->block_bytes, cudaMemcpyHostToDevice));
        else PIE_CUDA(cudaMemcpy(host_buf, p, (size_t)pool->block_bytes, cudaMemcpyDeviceToHost));
    } else {
        if (write) std::memcpy(p, host_buf, (size_t)pool->block_bytes);
        else std::memcpy(host_buf, p, (size_t)pool->block_bytes);
    }
    return PIE_OK;
}

int pie_block_write(pie_pool *pool, int32_t layer, int32_t block, const void *host_buf) {
    return unit_access(pool, layer, block, const_cast<void *>(host_buf), true);
}
int pie_block_read(pie_pool *pool, int32_t layer, int32_t block, void *host_buf) {
    return unit_access(pool, layer, block, host_buf, false);
}

int pie_block_state(pie_pool *pool, int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot, int32_t *host_slot) {
    if (!pool) return PIE_ERR_INVALID;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    return pool->table->state(layer, block, state, gpu_slot, host_slot);
}

int pie_get_placement(pie_pool *pool, int32_t *side, int32_t *slot) {
    if (!pool || !side || !slot) return PIE_ERR_INVALID;
    const int64_t n = (int64_t)pool->cfg.n_layers * pool->cfg.n_logical_blocks;
    for (int64_t i = 0; i < n; ++i) {
        const pie::Unit &u = pool->table->unit((int32_t)(i / pool->cfg.n_logical_blocks), (int32_t)(i % pool->cfg.n_logical_blocks));
        side[i] = u.side;
        slot[i] = u.side == PIE_GPU ? u.gpu_slot : u.side == PIE_HOST ? u.host_slot : -1;
    }
    return PIE_OK;
}

int pie_swap_out(pie_pool *pool, int32_t layer, const int32_t *block_ids, int64_t n, int32_t mode) {
    return pool_swap(pool, PIE_Q_OUT, layer, block_ids, n, mode);
}
int pie_swap_in(pie_pool *pool, int32_t layer, const int32_t *block_ids, int64_t n, int32_t mode) {
    return pool_swap(pool, PIE_Q_IN, layer, block_ids, n, mode);
}

int pie_swap_raw(pie_pool *pool, int32_t dir, const int32_t *src_slots, const int32_t *dst_slots, int64_t n, int32_t mode,
                 void *stream) {
    if (!pool || n < 0 || (n > 0 && (!src_slots || !dst_slots))) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (dir != PIE_H2D && dir != PIE_D2H) return PIE_ERR_INVALID;
    if (mode < PIE_MODE_AUTO || mode > PIE_MODE_KERNEL_BULK) return PIE_ERR_INVALID;
    const int64_t n_src = dir == PIE_H2D ? pool->cfg.n_host_slots : pool->cfg.n_gpu_slots;
    const int64_t n_dst = dir == PIE_H2D ? pool->cfg.n_gpu_slots : pool->cfg.n_host_slots;
    for (int64_t i = 0; i < n; ++i)
        if (src_slots[i] < 0 || src_slots[i] >= n_src || dst_slots[i] < 0 || dst_slots[i] >= n_dst) return PIE_ERR_RANGE;
    {
        std::vector<int32_t> sorted(dst_slots, dst_slots + n);
        std::sort(sorted.begin(), sorted.end());
        if (std::adjacent_find(sorted.begin(), sorted.end()) != sorted.end()) return PIE_ERR_INVALID;
    }
    if (n == 0) return PIE_OK;
    const int queue = dir == PIE_H2D ? PIE_Q_IN : PIE_Q_OUT;
    cudaStream_t s = stream ? (cudaStream_t)stream : pool->stream[queue];
    int st = do_copies(pool, queue, src_slots, dst_slots, n, nullptr, nullptr, mode, s);
    if (st == PIE_OK) (queue == PIE_Q_IN ? pool->stats.bytes_in : pool->stats.bytes_out) += (double)n * (double)pool->block_bytes;
    return st;
}

int pie_decode_attention(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                         int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, const int32_t *block_table_host,
                         const int32_t *ctx_lens_host, int32_t n_seqs, float scale, const void *k_new, const void *v_new) {
    return attention_call(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, block_table_host,
                          ctx_lens_host, n_seqs, scale, k_new, v_new);
}

// Evaluate one step's event set: per-layer compute, stall and swap times -> stats -> (adaptive mode) the ratio.
// wait = true blocks until the set's events have completed (used only when the ring is about to wrap).
static int evaluate_step_set(pie_pool *pool, int k, bool wait, int32_t *changed) {
    std::vector<LayerEvents> &ev = pool->lev[k];
    if (!pool->lev_closed[k]) {
        // the set's newest compute ticket has no mark yet (a caller that went layer by layer and never ticked)
        if (!wait) return 1;
        const size_t set_words = (size_t)pool->cfg.n_layers * STAMP_WORDS;
        PIE_CUDA(cudaMemcpyAsync(pool->stamps_host + (size_t)k * set_words, pool->stamps_dev + (size_t)k * set_words, set_words * 8,
                                 cudaMemcpyDeviceToHost, pool->stream[PIE_Q_COMPUTE]));
        PIE_CUDA(cudaStreamSynchronize(pool->stream[PIE_Q_COMPUTE]));
        pool->lev_closed[k] = true;
    }
    // every event of the set sits on one of three streams and a stream completes in order: the newest event of
    // each stream tells whether the whole set is complete
    for (int q = 1; q <= 3; ++q) {
        cudaEvent_t evt = pool->lev_last[k][q];
        if (!evt) continue;
        if (wait) PIE_CUDA(cudaEventSynchronize(evt));
        else if (cudaEventQuery(evt) != cudaSuccess) return 1;  // not complete yet
    }
    double compute = 0, stall = 0, t_in = 0, t_out = 0;
    bool any_swap = false;
    const size_t L = ev.size();
    const volatile uint64_t *stamps = pool->stamps_host + (size_t)k * L * STAMP_WORDS;
    std::vector<float> dur_in(L, -1.f), dur_out(L, -1.f);
    for (size_t l = 0; l < L; ++l) {
        LayerEvents &e = ev[l];
        float ms = 0;
        if (e.has_in) {
            PIE_CUDA(cudaEventElapsedTime(&ms, e.in0, e.in1));
            t_in += ms;
            dur_in[l] = ms;
            any_swap = true;
        }
        if (e.has_out) {
            PIE_CUDA(cudaEventElapsedTime(&ms, e.out0, e.out1));
            t_out += ms;
            dur_out[l] = ms;
            any_swap = true;
        }
    }
    // Compute stream, from the GPU-timer stamps.  A layer's time runs from the end of the previous layer's attention
    // kernel to the end of its own (combine and launch gap included, with or without swaps).  What the gap before a
    // layer that had units brought in exceeds the usual gap by is the stall: the stream sat in the presence wait.  The
    // usual gap is the smallest one of the step, but no more than 20 us, so that a step in which every layer waits
    // still shows it - or the smallest gap of the newest swap-free step, where that is larger.
    const bool chained = pool->prev_step_id == pool->lev_step[k] - 1 && pool->prev_step_end != 0;
    uint64_t prev_end = chained ? pool->prev_step_end : 0, first = 0, last = 0;
    uint64_t usual_gap = 20000;
    double first_stall = 0.0;
    std::vector<double> spans;   // per layer but the step's first: end of the previous layer's kernel to the end of its own, less the wait
    {
        uint64_t pe = 0, step_min = ~uint64_t(0);
        for (size_t l = 0; l < L; ++l) {
            const uint64_t S = stamps[l * STAMP_WORDS + STAMP_START], E = stamps[l * STAMP_WORDS + STAMP_END];
            if (!ev[l].has_compute || !S || !E) continue;
            if (pe && S > pe) step_min = std::min(step_min, S - pe);
            pe = E;
        }
        // A caller that runs other kernels between the layers has long gaps without any waiting: the smallest gap of
        // the newest step that moved nothing is the better yardstick where one has been seen.
        if (!any_swap && step_min != ~uint64_t(0)) pool->free_step_gap_ns = step_min;
        if (pool->free_step_gap_ns) usual_gap = std::max(pool->free_step_gap_ns, std::min(usual_gap, step_min));
        else usual_gap = std::min(usual_gap, step_min);
    }
    for (size_t l = 0; l < L; ++l) {
        const uint64_t S = stamps[l * STAMP_WORDS + STAMP_START], E = stamps[l * STAMP_WORDS + STAMP_END];
        if (!ev[l].has_compute || !S || !E || E < S) continue;
        const bool fetched = ev[l].stream_wait;
        // the presence wait: what the kernel itself waited for the layer's arrival word, plus - where the stream had to
        // wait - what the gap before the kernel exceeds the usual gap by
        const double kernel_wait = (double)stamps[l * STAMP_WORDS + STAMP_WAIT] * 1e-6;
        double layer_stall = kernel_wait;
        if (fetched && prev_end && S > prev_end + usual_gap) layer_stall += (double)(S - prev_end - usual_gap) * 1e-6;
        stall += layer_stall;

        if (!first) {
            // the step's first layer: its time starts with its own kernel (whatever the caller did between two steps
            // is not the layer's); a wait before it still counts as stall, and as part of the step
            first = S;
            first_stall = layer_stall - kernel_wait;   // the wait inside the kernel is part of E - S already
            compute += std::max(0.0, (double)(E - S) * 1e-6 - (double)stamps[l * STAMP_WORDS + STAMP_WAIT] * 1e-6);
        } else {
            const double span = std::max(0.0, (double)(E - prev_end) * 1e-6 - layer_stall);
            compute += span;
            spans.push_back(span);
        }
        prev_end = last = E;
    }
    if (last) {
        pool->prev_step_end = last;
        pool->prev_step_id = pool->lev_step[k];
    }
    pool->lev_done[k] = true;
    if (first && pool->cfg.timing >= 2) {
        // compute columns from the stamps, relative to the first kernel's start; copy columns from the copy streams'
        // events relative to the step's anchor event, which was recorded just before that kernel
        pool->timeline.assign(L * 7, -1.f);
        auto rel = [&](uint64_t t) { return (float)(((double)t - (double)first) * 1e-6); };
        uint64_t before = first;
        for (size_t l = 0; l < L; ++l) {
            const uint64_t S = stamps[l * STAMP_WORDS + STAMP_START], E = stamps[l * STAMP_WORDS + STAMP_END];
            float *row = pool->timeline.data() + l * 7;
            if (ev[l].has_compute && S && E) {
                row[0] = rel(before);
                row[1] = rel(S + stamps[l * STAMP_WORDS + STAMP_WAIT]);   // past the presence wait inside the kernel
                row[2] = rel(E);
                before = E;
            }
            if (!pool->lev_anchored[k]) continue;
            float ms = 0;
            if (ev[l].has_in && cudaEventElapsedTime(&ms, pool->lev_anchor[k], ev[l].in0) == cudaSuccess) {
                row[3] = ms;
                row[4] = ms + dur_in[l];
            }
            if (ev[l].has_out && cudaEventElapsedTime(&ms, pool->lev_anchor[k], ev[l].out0) == cudaSuccess) {
                row[5] = ms;
                row[6] = ms + dur_out[l];
            }
        }
    }
    pool->stats.last_step_compute_ms = compute;
    pool->stats.last_step_stall_ms = stall;
    pool->stats.last_step_swap_in_ms = t_in;
    pool->stats.last_step_swap_out_ms = t_out;
    if (first && last) pool->stats.last_step_ms = (double)(last - first) * 1e-6 + first_stall;
    pool->stats.steps_measured += 1;
    pool->stats.last_step_violation_ratio =
        pool->step_prefetch[k][0] > 0 ? (double)pool->step_prefetch[k][1] / (double)pool->step_prefetch[k][0] : 0.0;
    // Copies that are hidden behind compute can still slow the compute down (they share HBM); that excess counts as a
    // wait, so the controller holds the ratio where wait + slow-down stays within its tolerance.  Every layer of a step
    // attends the same batch at the same lengths, and the swap lists of a group of layers are in flight during the first
    // part of the group only: the step's undisturbed layers are its own yardstick.  The contrast of a series of layer
    // times = what they add up to above the mean of the series' fastest quarter, over their sum.  Consecutive launches
    // overlap at their ends, so the end stamp of a layer moves by a few per cent of a layer from one to the next (what one
    // layer's time gains the next one's loses) while copies slow several layers in a row: the slow-down is the contrast
    // of the four-layer means, less the larger of what that comes to on steps without swap traffic (a record,
    // Section 3.4.2) and 0.3 of the contrast of the single layers (measured: alternating end stamps pass a four-layer
    // mean at a quarter of their size).  Nothing is compared across steps, so clocks drifting under the power cap and
    // contexts growing do not look like a slow-down.  (Steps of fewer than nine layers fall back to a record of the
    // time per context token taken on swap-free steps.)
    double tokens = 0.0;   // the step's own count (each kernel notes its batch's tokens beside its time stamps)
    for (size_t l = 0; l < L && tokens == 0.0; ++l)
        if (ev[l].has_compute) tokens = (double)stamps[l * STAMP_WORDS + STAMP_TOKENS];
    double slow = 0.0;
    if (spans.size() >= 8 && compute > 0) {
        auto contrast = [](const std::vector<double> &v) {
            std::vector<double> sorted(v);
            std::sort(sorted.begin(), sorted.end());
            const size_t quarter = std::max<size_t>(2, sorted.size() / 4);
            double ref = 0.0, sum = 0.0, above = 0.0;
            for (size_t i = 0; i < quarter; ++i) ref += sorted[i];
            ref /= (double)quarter;
            for (double x : v) {
                sum += x;
                above += std::max(0.0, x - ref);
            }
            return sum > 0 ? above / sum : 0.0;
        };
        std::vector<double> means(spans.size() - 3);
        for (size_t i = 0; i + 3 < spans.size(); ++i) means[i] = 0.25 * (spans[i] + spans[i + 1] + spans[i + 2] + spans[i + 3]);
        const double smooth = contrast(means);
        if (!any_swap) pool->free_contrast = pool->free_contrast >= 0 ? 0.75 * pool->free_contrast + 0.25 * smooth : smooth;
        else slow = std::max(0.0, smooth - std::max(std::max(0.0, pool->free_contrast), 0.3 * contrast(spans))) * compute;
    } else if (tokens > 0 && compute > 0) {
        const double per_token = compute / tokens;
        if (!any_swap) pool->base_ms_per_token = pool->base_ms_per_token > 0 ? 0.75 * pool->base_ms_per_token + 0.25 * per_token : per_token;
        else if (pool->base_ms_per_token > 0) slow = std::max(0.0, compute - pool->base_ms_per_token * tokens);
    }
    pool->stats.last_step_slowdown_ms = slow;
    pool->stats.ratio_floor = ratio_floor(pool);
    if (pool->ratio_mode == 2 && compute > 0) {
        const double step = pool->ctrl_step > 0 ? pool->ctrl_step : 1.0 / (double)pool->cfg.n_layers;  // "one layer" (Section 3.4.2)
        // the rule never asks for less than the GPU pool's size allows: below that floor the number would drift
        // away from what the layers actually keep on the host
        const double r = std::max(ratio_floor(pool),
                                  std::min(pool->ratio_cap, pie_controller_decide(pool->ctrl_state, pool->ratio, step, stall + slow,
                                                                                  compute, std::max(t_in, t_out))));
        if (r != pool->ratio) {
            pool->ratio = r;
            if (changed) *changed = 1;
        }
    }
    return PIE_OK;
}

// evaluate, in step order, every completed set that has not been evaluated yet
static int evaluate_completed(pie_pool *pool, int32_t *changed) {
    // (the step in progress counts once its set has been closed: pie_controller_tick after the last layer)
    for (int64_t st = std::max<int64_t>(1, pool->step - TIMING_RING + 1); st <= pool->step; ++st) {
        const int k = (int)(st % TIMING_RING);
        if (pool->lev_step[k] != st || pool->lev_done[k]) continue;
        const int rc = evaluate_step_set(pool, k, false, changed);
        if (rc < 0) return rc;
        if (rc == 1) break;  // this one is still running: so are the later ones
    }
    return PIE_OK;
}

int pie_step_begin(pie_pool *pool) {
    if (!pool) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;   // (a launch that failed stores no ticket: nothing may wait for one)
    {
        int st = finish_group(pool);       // a caller that went layer by layer may have left a group open
        if (st == PIE_OK) st = close_step_set(pool);
        if (st == PIE_OK) st = mark_step_end(pool);
        if (st != PIE_OK) return st;
    }
    ++pool->step;
    if (pool->step >= 2 + pool->run_ahead) {   // run_ahead steps (two, by default) ahead of the GPU at most (mark_step_end)
        const int64_t old = pool->step - 1 - pool->run_ahead;
        const int k = (int)(old % TIMING_RING);
        if (pool->step_end_of[k] == old) PIE_CUDA(cudaEventSynchronize(pool->step_end_ev[k]));
    }
    if (pool->cfg.timing) {
        int st = evaluate_completed(pool, nullptr);
        if (st != PIE_OK) return st;
        const int k = (int)(pool->step % TIMING_RING);
        if (pool->lev_step[k] != 0 && !pool->lev_done[k]) {
            // the ring wraps: the host is TIMING_RING steps ahead of the GPU; wait for that step and evaluate it
            st = evaluate_step_set(pool, k, true, nullptr);
            if (st < 0) return st;
        }
        pool->lev_step[k] = pool->step;
        pool->lev_done[k] = false;
        pool->lev_closed[k] = true;    // no compute ticket in the set yet
        for (LayerEvents &e : pool->lev[k]) e.has_in = e.has_out = e.has_compute = e.stream_wait = false;
        for (int q = 0; q < 4; ++q) pool->lev_last[k][q] = nullptr;
        pool->lev_anchored[k] = false;
        pool->step_prefetch[k][0] = pool->step_prefetch[k][1] = 0;
        // the set's kernels are launched after this point, and the previous user of the set has completed
        std::memset(pool->stamps_host + (size_t)k * (size_t)pool->cfg.n_layers * STAMP_WORDS, 0,
                    (size_t)pool->cfg.n_layers * STAMP_WORDS * 8);
    }
    return PIE_OK;
}

int pie_set_extension_ratio(pie_pool *pool, float r) {
    if (!pool || r > 1.0f || r != r) return PIE_ERR_INVALID;
    if (r < 0.f) {
        if (!pool->cfg.timing) return PIE_ERR_INVALID;  // the controller needs the per-layer events
        if (pool->ratio_mode == 0) {
            // the controller takes over from the sets the caller established (all on the GPU gives 0: the paper's
            // starting point, Section 3.4.2)
            float cur = 0.f;
            pie_get_extension_ratio(pool, &cur);
            pool->ratio = cur;
        }
        pool->ratio_mode = 2;
    } else {
        pool->ratio_mode = 1;
        pool->ratio = r;
    }
    return PIE_OK;
}

int pie_set_controller(pie_pool *pool, double step, double eps, double u_hi) {
    if (!pool || step > 1.0 || eps >= 1.0 || u_hi > 1.0) return PIE_ERR_INVALID;
    if (step > 0) pool->ctrl_step = step;
    if (eps > 0) pool->ctrl_state[5] = eps;
    if (u_hi > 0) pool->ctrl_state[6] = u_hi;
    return PIE_OK;
}

int pie_get_extension_ratio(pie_pool *pool, float *r) {
    if (!pool || !r) return PIE_ERR_INVALID;
    if (pool->ratio_mode == 0) {
        int64_t home = 0;
        for (int64_t c : pool->home_count) home += c;
        const int64_t units = (int64_t)pool->table->n_allocated() * pool->cfg.n_layers;
        *r = units > 0 ? (float)((double)home / (double)units) : 0.f;
    } else {
        *r = (float)pool->ratio;
    }
    return PIE_OK;
}

int pie_kv_write(pie_pool *pool, int32_t layer, const void *k, const void *v, const int32_t *token_seq_dev,
                 const int32_t *token_pos_dev, int64_t n_tokens, const int32_t *block_table_dev, int32_t max_blocks_per_seq,
                 int32_t n_seqs) {
    if (!pool || n_tokens < 0 || max_blocks_per_seq <= 0 || n_seqs <= 0) return PIE_ERR_INVALID;
    if (n_tokens > 0 && (!k || !v || !token_seq_dev || !token_pos_dev || !block_table_dev)) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (layer < 0 || layer >= pool->cfg.n_layers) return PIE_ERR_RANGE;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    st = check_status_word(pool);
    if (st != PIE_OK) return st;
    if (n_tokens == 0) return PIE_OK;
    // like an attention call: a compute ticket, behind every copy that is still bringing a unit of the layer in
    int64_t ticket = 0, waits[4];
    st = pool->table->attention(layer, nullptr, 0, &ticket, waits);
    if (st != PIE_OK) return st;
    if (pool->table->tracks_writes()) pool->table->mark_layer_dirty(layer);  // which blocks are written is on the device only
    cudaStream_t stream = pool->stream[PIE_Q_COMPUTE];
    st = reserve_ticket_event(pool, PIE_Q_COMPUTE, ticket);
    if (st != PIE_OK) { pool->sticky = st; return st; }
    for (int qd = 1; qd <= 2; ++qd) {
        st = wait_ticket(pool, stream, qd, waits[qd]);
        if (st != PIE_OK) { pool->sticky = st; return st; }
    }
    const int32_t *slots = pool->slot_table_dev + (int64_t)layer * pool->cfg.n_logical_blocks;
    cudaError_t e = pool->kv_fp8
                        ? pie::launch_kv_write8(k, v, token_seq_dev, token_pos_dev, n_tokens, block_table_dev, max_blocks_per_seq, n_seqs,
                                                slots, pool->cfg.n_logical_blocks, pool->cfg.n_gpu_slots, pool->gpu_base,
                                                pool->cfg.n_kv_heads, pool->cfg.dtype, pool->k_scale, pool->v_scale, pool->status_dev, stream)
                        : pie::launch_kv_write(k, v, token_seq_dev, token_pos_dev, n_tokens, block_table_dev, max_blocks_per_seq, n_seqs,
                                               slots, pool->cfg.n_logical_blocks, pool->cfg.n_gpu_slots, pool->gpu_base,
                                               pool->cfg.n_kv_heads, pool->cfg.head_dim, pool->status_dev, stream);
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        pool->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    st = record_ticket(pool, PIE_Q_COMPUTE, ticket);
    if (st != PIE_OK) pool->sticky = st;
    return st;
}

int pie_prefill_attention(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                          int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, const int32_t *q_offsets_dev,
                          const int32_t *ctx_lens_host, const int32_t *q_offsets_host, int32_t n_seqs, float scale) {
    if (!pool || !q || !out || !block_table_dev || !ctx_lens_dev || !q_offsets_dev || !ctx_lens_host || !q_offsets_host)
        return PIE_ERR_INVALID;
    if (n_seqs < 0 || max_blocks_per_seq <= 0) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (pool->kv_fp8) return PIE_ERR_UNSUPPORTED;
    if (layer < 0 || layer >= pool->cfg.n_layers) return PIE_ERR_RANGE;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    st = check_status_word(pool);
    if (st != PIE_OK) return st;
    if (n_seqs == 0) return PIE_OK;
    // a chunk is at most its context, which is at most the table; 128 query rows per tile = 128 / G tokens
    const int32_t G = pool->cfg.n_q_heads / pool->cfg.n_kv_heads, tile_tokens = 128 / G;
    if (q_offsets_host[0] != 0) return PIE_ERR_INVALID;
    int64_t n_tiles = 0;
    for (int32_t s = 0; s < n_seqs; ++s) {
        const int64_t c = (int64_t)q_offsets_host[s + 1] - q_offsets_host[s];
        if (c < 0 || ctx_lens_host[s] < 0 || c > ctx_lens_host[s] || ctx_lens_host[s] > max_blocks_per_seq * 16) return PIE_ERR_INVALID;
        n_tiles += (c + tile_tokens - 1) / tile_tokens;
    }
    if (n_tiles * pool->cfg.n_kv_heads > 0x7fffffffll) return PIE_ERR_INVALID;
    if (n_tiles == 0) return PIE_OK;
    if (!pool->prefill_ready) {
        PIE_CUDA(pie::prefill_configure(pool->cfg.head_dim, pool->cfg.dtype));
        pool->prefill_ready = true;
    }
    // like an attention call: a compute ticket, behind every copy that is still bringing a unit of the layer in
    int64_t ticket = 0, waits[4];
    st = pool->table->attention(layer, nullptr, 0, &ticket, waits);
    if (st != PIE_OK) return st;
    cudaStream_t stream = pool->stream[PIE_Q_COMPUTE];
    for (int qd = 1; qd <= 2; ++qd) {
        st = wait_ticket(pool, stream, qd, waits[qd]);
        if (st != PIE_OK) { pool->sticky = st; return st; }
    }
    // the tiles' prefix sums go to the device through the list ring
    int64_t off = 0;
    st = list_alloc(pool, n_seqs + 1, &off);
    if (st != PIE_OK) { pool->sticky = st; return st; }
    int32_t *h = pool->list_host + off;
    h[0] = 0;
    for (int32_t s = 0; s < n_seqs; ++s)
        h[s + 1] = h[s] + (q_offsets_host[s + 1] - q_offsets_host[s] + tile_tokens - 1) / tile_tokens;
    cudaError_t e = cudaMemcpyAsync(pool->list_dev + off, h, (size_t)(n_seqs + 1) * 4, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) {
        pie::AttnShape sh{pool->cfg.head_dim, pool->cfg.dtype, pool->cfg.n_q_heads, pool->cfg.n_kv_heads, pool->cfg.n_logical_blocks,
                          pool->cfg.n_gpu_slots, 0};
        pie::PrefillLaunch a{};
        a.q = q;
        a.out = out;
        a.block_table = block_table_dev;
        a.max_blocks = max_blocks_per_seq;
        a.ctx_lens = ctx_lens_dev;
        a.q_offsets = q_offsets_dev;
        a.tile_off = pool->list_dev + off;
        a.slot_table = pool->slot_table_dev + (int64_t)layer * pool->cfg.n_logical_blocks;
        a.n_seqs = n_seqs;
        a.n_tiles = (int32_t)n_tiles;
        a.scale = scale;
        a.status = pool->status_dev;
        e = pie::launch_prefill_attention(sh, a, pool->map_prefill, stream);
    }
    if (e != cudaSuccess) {
        g_last_cuda_error = (int)e;
        pool->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    st = list_commit(pool, off, n_seqs + 1, stream);
    if (st == PIE_OK) st = record_ticket(pool, PIE_Q_COMPUTE, ticket);
    if (st != PIE_OK) pool->sticky = st;
    return st;
}

int pie_report_throughput(pie_pool *pool, double throughput) {
    if (!pool || !std::isfinite(throughput) || throughput < 0) return PIE_ERR_INVALID;
    const double step = pool->ctrl_step > 0 ? pool->ctrl_step : 1.0 / (double)pool->cfg.n_layers;
    if (!pool->governor) {
        pool->governor = pie_governor_create(step, 0, 0, 0);
        if (!pool->governor) return PIE_ERR_NOMEM;
    }
    pool->ratio_cap = pie_governor_report(pool->governor, pool->ratio, throughput);
    int32_t state = 0;
    pie_governor_state(pool->governor, &state, nullptr);
    pool->stats.governor_cap = pool->ratio_cap;
    pool->stats.governor_state = (uint32_t)state;
    return PIE_OK;
}

int pie_set_kv_scales(pie_pool *pool, float k_scale, float v_scale) {
    if (!pool || !(k_scale > 0.f) || !(v_scale > 0.f) || !std::isfinite(k_scale) || !std::isfinite(v_scale)) return PIE_ERR_INVALID;
    if (!pool->kv_fp8) return PIE_ERR_UNSUPPORTED;
    pool->k_scale = k_scale;
    pool->v_scale = v_scale;
    return PIE_OK;
}

int pie_set_lookahead(pie_pool *pool, int32_t layers) {
    if (!pool || layers < 0 || layers > MAX_GROUP_LAYERS) return PIE_ERR_INVALID;
    int st = finish_group(pool);
    if (st != PIE_OK) return st;
    pool->group_setting = layers;
    pool->lookahead = std::max(1, layers);
    return PIE_OK;
}

int pie_set_run_ahead(pie_pool *pool, int32_t steps) {
    if (!pool || steps < 1 || steps > TIMING_RING - 1) return PIE_ERR_INVALID;
    pool->run_ahead = steps;
    return PIE_OK;
}

int pie_set_retention(pie_pool *pool, int32_t on) {
    if (!pool) return PIE_ERR_INVALID;
    pool->table->set_retain(on != 0);
    return PIE_OK;
}

int pie_declare_append_blocks(pie_pool *pool, const int32_t *ids, int64_t n) {
    if (!pool || (n > 0 && !ids)) return PIE_ERR_INVALID;
    if (n < 0) {
        pool->append_declared = false;
        pool->append_ids.clear();
        return PIE_OK;
    }
    for (int64_t i = 0; i < n; ++i)
        if (ids[i] < 0 || ids[i] >= pool->cfg.n_logical_blocks) return PIE_ERR_RANGE;
    pool->append_ids.assign(ids, ids + n);
    pool->append_declared = true;
    return PIE_OK;
}

int pie_resize_begin(pie_pool *pool, int32_t new_blocks) {
    if (!pool) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    return pool->table->resize_begin(new_blocks);
}

int pie_resize_status(pie_pool *pool, int32_t *visible, int32_t *alloc_limit, int32_t *target, int32_t *layers_moved) {
    if (!pool) return PIE_ERR_INVALID;
    if (visible) *visible = pool->table->capacity();
    if (alloc_limit) *alloc_limit = pool->table->alloc_limit();
    if (target) *target = pool->table->resize_target();
    if (layers_moved) *layers_moved = pool->table->layers_moved();
    return PIE_OK;
}

int pie_plan_layer(pie_pool *pool, int32_t layer, int32_t *in_ids, int64_t *n_in, int32_t *out_ids, int64_t *n_out) {
    if (!pool || !in_ids || !n_in || !out_ids || !n_out) return PIE_ERR_INVALID;
    if (layer < 0 || layer >= pool->cfg.n_layers) return PIE_ERR_RANGE;
    int st = poll(pool);
    if (st != PIE_OK) return st;
    plan_layer(pool, layer, pool->v_in, pool->v_out);
    std::copy(pool->v_in.begin(), pool->v_in.end(), in_ids);
    std::copy(pool->v_out.begin(), pool->v_out.end(), out_ids);
    *n_in = (int64_t)pool->v_in.size();
    *n_out = (int64_t)pool->v_out.size();
    return PIE_OK;
}

int pie_controller_tick(pie_pool *pool, int32_t *changed) {
    if (!pool) return PIE_ERR_INVALID;
    if (changed) *changed = 0;
    int st = finish_group(pool);
    if (st != PIE_OK) return st;
    if (!pool->cfg.timing) return PIE_OK;
    st = close_step_set(pool);
    if (st != PIE_OK) return st;
    return evaluate_completed(pool, changed);
}

int pie_get_step_timeline(pie_pool *pool, float *ms, int64_t capacity) {
    if (!pool || !ms) return PIE_ERR_INVALID;
    if ((int64_t)pool->timeline.size() > capacity || pool->timeline.empty()) return PIE_ERR_INVALID;
    std::copy(pool->timeline.begin(), pool->timeline.end(), ms);
    return PIE_OK;
}

int pie_get_stats(pie_pool *pool, pie_stats *out_caller) {
    if (!pool || !out_caller) return PIE_ERR_INVALID;
    if (out_caller->struct_size < offsetof(pie_stats, steps_measured) + sizeof(int64_t)) return PIE_ERR_INVALID;
    // filled in a struct of this build's layout, then as much of it copied out as the caller's struct holds
    struct Copy {
        pie_stats local;
        pie_stats *dst;
        ~Copy() {
            const uint32_t n = std::min<uint32_t>(dst->struct_size, (uint32_t)sizeof local);
            local.struct_size = dst->struct_size;
            std::memcpy(dst, &local, n);
        }
    } copy{pool->stats, out_caller};
    pie_stats *out = &copy.local;
    poll(pool);
    float r = 0;
    pie_get_extension_ratio(pool, &r);
    out->ratio = r;
    int64_t g = 0, h = 0, f = 0;
    const int64_t n = (int64_t)pool->cfg.n_layers * pool->cfg.n_logical_blocks;
    for (int64_t i = 0; i < n; ++i) {
        const pie::Unit &u = pool->table->unit((int32_t)(i / pool->cfg.n_logical_blocks), (int32_t)(i % pool->cfg.n_logical_blocks));
        if (u.side == PIE_FREE) continue;
        if (pool->table->in_flight(u)) ++f;
        else if (u.side == PIE_GPU) ++g;
        else ++h;
    }
    out->n_units_gpu = g;
    out->n_units_host = h;
    out->n_units_in_flight = f;
    return PIE_OK;
}

int pie_sync(pie_pool *pool, int64_t timeout_us) {
    if (!pool) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    int st = finish_group(pool);
    if (st != PIE_OK) return st;
    st = sync_all(pool, timeout_us);
    if (st != PIE_OK) return st;
    return check_status_word(pool);
}

// ---- whole-layer protocol on the GPU ------------------------------------------------------------------------
static void all_block_ids(pie_pool *pool, std::vector<int32_t> &ids) {
    ids.clear();
    for (int32_t b = 0; b < pool->cfg.n_logical_blocks; ++b)
        if (pool->table->allocated(b)) ids.push_back(b);
}

int pie_set_layer_policy(pie_pool *pool, int32_t gpu_regions, int32_t cpu_regions) {
    if (!pool) return PIE_ERR_INVALID;
    if (gpu_regions <= 0 && cpu_regions <= 0) {  // back to the block-granular plan
        delete pool->fifo;
        pool->fifo = nullptr;
        return PIE_OK;
    }
    const int32_t L = pool->cfg.n_layers;
    if (gpu_regions <= 0 || cpu_regions < 0 || gpu_regions + cpu_regions < L) return PIE_ERR_INVALID;
    int st = finish_group(pool);
    if (st != PIE_OK) return st;
    st = sync_all(pool, 30 * 1000 * 1000);  // layers must be settled, each wholly on one side
    if (st != PIE_OK) return st;
    std::vector<uint8_t> on_cpu((size_t)L, 0);
    int32_t n_gpu = 0, n_cpu = 0;
    for (int32_t l = 0; l < L; ++l) {
        int64_t g = 0, h = 0;
        for (int32_t b = 0; b < pool->cfg.n_logical_blocks; ++b) {
            if (!pool->table->allocated(b)) continue;
            (pool->table->unit(l, b).side == PIE_GPU ? g : h) += 1;
        }
        if (g > 0 && h > 0) return PIE_ERR_INVALID;  // a layer split between the sides: not a whole-layer state
        on_cpu[(size_t)l] = h > 0;
        (h > 0 ? n_cpu : n_gpu) += 1;
    }
    if (n_gpu > gpu_regions || n_cpu > cpu_regions) return PIE_ERR_NOMEM;
    delete pool->fifo;
    pool->fifo = new (std::nothrow) pie::Fifo(L, gpu_regions, cpu_regions, on_cpu.data());
    if (!pool->fifo) return PIE_ERR_NOMEM;
    pool->fifo_ticket[PIE_Q_IN] = pool->fifo_ticket[PIE_Q_OUT] = 0;
    pool->fifo_cpu_layers = std::max(0, cpu_regions - 2);
    pool->fifo_log.clear();
    return PIE_OK;
}

// Whole-layer mode with m layers on the CPU: n - m GPU regions and m + 2 CPU regions (Section 3.3).  Between two
// tokens: everything settles, as many whole layers as the new region counts require move (the coldest GPU layers out -
// the highest, seen from layer 0 - or the hottest CPU layers in), and the scheduler starts afresh from the placement.
static int fifo_set_cpu_layers(pie_pool *pool, int32_t m, int32_t mode) {
    const int32_t L = pool->cfg.n_layers;
    m = std::max(0, std::min(m, L - 2));
    std::vector<int32_t> ids;
    all_block_ids(pool, ids);
    for (int pass = 0; pass < 2 * L; ++pass) {
        int st = sync_all(pool, 30 * 1000 * 1000);
        if (st != PIE_OK) return st;
        std::vector<int32_t> on_gpu, on_cpu;
        for (int32_t l = 0; l < L; ++l) {
            bool host = false;
            for (int32_t b : ids) host = host || pool->table->unit(l, b).side == PIE_HOST;
            (host ? on_cpu : on_gpu).push_back(l);
        }
        if ((int32_t)on_gpu.size() > L - m) st = pool_swap(pool, PIE_Q_OUT, on_gpu.back(), ids.data(), (int64_t)ids.size(), mode);
        else if ((int32_t)on_cpu.size() > m + 2) st = pool_swap(pool, PIE_Q_IN, on_cpu.front(), ids.data(), (int64_t)ids.size(), mode);
        else break;
        if (st != PIE_OK) return st;
    }
    std::vector<int32_t> log;
    log.swap(pool->fifo_log);            // the decisions so far stay readable across the change
    const int st = pie_set_layer_policy(pool, L - m, m + 2);
    pool->fifo_log.swap(log);
    return st;
}

int pie_set_violation_trigger(pie_pool *pool, double share) {
    if (!pool || share < 0 || share > 1 || share != share) return PIE_ERR_INVALID;
    pool->violation_trigger = share;
    return PIE_OK;
}

int pie_get_layer_log(pie_pool *pool, int32_t *log, int64_t capacity, int64_t *n_entries) {
    if (!pool || !n_entries) return PIE_ERR_INVALID;
    const int64_t n = (int64_t)pool->fifo_log.size() / 4;
    *n_entries = n;
    if (log) {
        if (capacity < n * 4) return PIE_ERR_INVALID;
        std::copy(pool->fifo_log.begin(), pool->fifo_log.end(), log);
    }
    return PIE_OK;
}

// A swap-in list started by the decode loop; next_token: it serves a layer that only the next token needs (Section
// 3.4.2's allowed rule violation: the prefetch that wraps around the last layer).
static void count_prefetch(pie_pool *pool, bool next_token) {
    pool->stats.prefetch_lists += 1;
    pool->stats.prefetch_violations += next_token;
    const int k = (int)(pool->step % TIMING_RING);
    pool->step_prefetch[k][0] += 1;
    pool->step_prefetch[k][1] += next_token;
}

// confirmed completions -> scheduler (a finished swap-out frees its GPU region, a finished swap-in its CPU region)
static int fifo_apply_completions(pie_pool *pool) {
    int st = poll(pool);
    if (st != PIE_OK) return st;
    for (int q : {PIE_Q_OUT, PIE_Q_IN})
        if (pool->fifo_ticket[q] > 0 && pool->fifo_ticket[q] <= pool->table->done(q)) {
            pool->fifo->complete(q);
            pool->fifo_ticket[q] = 0;
        }
    return PIE_OK;
}

// the protocol's step at the instant layer k starts: start the swaps the scheduler asks for
static int fifo_start_swaps(pie_pool *pool, int32_t k, int32_t mode, std::vector<int32_t> &ids) {
    int32_t so = -1, si = -1;
    int st = pool->fifo->layer_start(k, &so, &si);
    if (st != PIE_OK) return st;
    pool->fifo_log.insert(pool->fifo_log.end(), {(int32_t)pool->step, k, so, si});
    if (si >= 0) count_prefetch(pool, si < k);
    for (int which = 0; which < 2; ++which) {
        const int32_t layer = which == 0 ? so : si;
        const int q = which == 0 ? PIE_Q_OUT : PIE_Q_IN;
        if (layer < 0) continue;
        all_block_ids(pool, ids);
        const int64_t before = pool->table->issued(q);
        st = pool_swap(pool, q, layer, ids.data(), (int64_t)ids.size(), mode);
        if (st != PIE_OK) return st;
        // an empty layer moves nothing and is complete at once
        if (pool->table->issued(q) == before) pool->fifo->complete(q);
        else pool->fifo_ticket[q] = pool->table->issued(q);
    }
    return PIE_OK;
}

static int decode_step_layers(pie_pool *pool, const void *q_all, void *out_all, const int32_t *block_table_dev,
                              int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, int32_t n_seqs, float scale,
                              const void *k_new_all, const void *v_new_all, int32_t mode) {
    const int32_t L = pool->cfg.n_layers;
    const int64_t q_stride = (int64_t)n_seqs * pool->cfg.n_q_heads * pool->cfg.head_dim * 2;
    const int64_t kv_stride = (int64_t)n_seqs * pool->cfg.n_kv_heads * pool->cfg.head_dim * 2;
    int st = pie_step_begin(pool);
    if (st != PIE_OK) return st;
    std::vector<int32_t> ids;
    const auto t_step = std::chrono::steady_clock::now();
    double waited_ms = 0.0;   // host clock: what the presence check below had to wait for layers still on the CPU
    for (int32_t k = 0; k < L; ++k) {
        // the control logic runs when layer k starts, i.e. when layer k-1 has finished: the host keeps step with
        // the device here (as the paper's per-layer control loop does), so completions are what they really are
        {
            cudaEvent_t prev_ev = nullptr;
            st = compute_mark(pool, pool->recorded[PIE_Q_COMPUTE], &prev_ev);
            if (st != PIE_OK) return st;
            if (prev_ev) PIE_CUDA(cudaEventSynchronize(prev_ev));
        }
        st = fifo_apply_completions(pool);
        if (st != PIE_OK) return st;
        st = fifo_start_swaps(pool, k, mode, ids);
        if (st != PIE_OK) return st;
        // presence check (Section 3.2): a layer still on the CPU with no copy under way has to be fetched first
        for (int guard = 0; pool->fifo->location(k) == 1; ++guard) {
            if (guard > 4 * L) return PIE_ERR_TIMEOUT;
            bool waited = false;
            const auto t_wait = std::chrono::steady_clock::now();
            for (int q : {PIE_Q_OUT, PIE_Q_IN})
                if (pool->fifo_ticket[q] > 0) {
                    PIE_CUDA(cudaEventSynchronize(pool->ticket_ev[q][pool->fifo_ticket[q] % EV_RING]));
                    waited = true;
                }
            waited_ms += std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t_wait).count();
            if (!waited) return PIE_ERR_NOMEM;  // nothing in flight and still no GPU region for layer k
            st = fifo_apply_completions(pool);
            if (st != PIE_OK) return st;
            st = fifo_start_swaps(pool, k, mode, ids);
            if (st != PIE_OK) return st;
        }
        // in transit to the GPU: the attention call waits for the copy's event on the device
        st = attention_call(pool, k, (const uint8_t *)q_all + k * q_stride, (uint8_t *)out_all + k * q_stride, block_table_dev,
                            max_blocks_per_seq, ctx_lens_dev, nullptr, nullptr, n_seqs, scale,
                            k_new_all ? (const uint8_t *)k_new_all + k * kv_stride : nullptr,
                            v_new_all ? (const uint8_t *)v_new_all + k * kv_stride : nullptr);
        if (st != PIE_OK) return st;
    }
    st = pie_controller_tick(pool, nullptr);
    if (st != PIE_OK || pool->ratio_mode != 2) return st;
    // Adaptive expansion in whole layers (Section 3.4.2): this token's waiting and the share of its swap-ins that were
    // for the next token decide how many layers live on the CPU from the next token on.
    const double step_ms = std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t_step).count();
    const int k_set = (int)(pool->step % TIMING_RING);
    const int32_t m = pool->fifo_cpu_layers;
    const int32_t m_new = pie_layer_controller_decide(pool->layer_ctrl_state, m, std::max(0, L - 2), waited_ms,
                                                      std::max(1e-9, step_ms - waited_ms), pool->step_prefetch[k_set][0],
                                                      pool->step_prefetch[k_set][1], pool->violation_trigger, pool->ctrl_state[5]);
    return m_new == m ? PIE_OK : fifo_set_cpu_layers(pool, m_new, mode);
}

// One layer of the control loop (Section 3.2; Section 4.2: what a model's forward pass calls per layer): fetch what the
// layer still lacks, attend (and append); at the start of a group of layers start the prefetch of the next group, at
// its end push the group's host-resident shares out.
static int decode_layer(pie_pool *pool, int32_t l, const void *q, void *out, const int32_t *block_table_dev,
                        int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, int32_t n_seqs, float scale, const void *k_new,
                        const void *v_new, int32_t mode, bool dependent = false, bool defer = false) {
    const int32_t L = pool->cfg.n_layers;
    struct PollHold {
        pie_pool *p;
        bool was;
        ~PollHold() { p->poll_hold = was; }
    } hold{pool, pool->poll_hold};
    // completions are learnt every few layers: a stale view only means a wait on an event that has already
    // completed, or a slot that stays "pending" a little longer
    if (l % 8 == 0) {
        int st = poll(pool, true);
        if (st != PIE_OK) return st;
    }
    pool->poll_hold = true;
    int st = PIE_OK;
    const bool continues = pool->group_len > 0 && l == pool->group_first + (int32_t)pool->group_done.size() &&
                           l < pool->group_first + pool->group_len;
    if (!continues) {
        // a new group starts with this layer (Section 3.3: the swaps are decided when a layer starts computing)
        st = finish_group(pool);
        if (st != PIE_OK) return st;
        const int32_t k = group_layers(pool);
        pool->group_first = l;
        pool->group_len = std::min(k, L - l);
        pool->group_mode = mode;
        // prefetch: the next group's layers (wrapping into the next token: the look-ahead of Section 3.4.2) that still
        // have units on the host.  The copies start when this group starts, i.e. once the previous attention call has
        // finished, and run back to back on the copy-in stream.  What the GPU pool cannot take now is fetched at
        // that layer's turn.
        const int32_t next_first = (l + pool->group_len) % L;
        const int32_t next_len = std::min(k, L - next_first);
        const int64_t start_with = pool->recorded[PIE_Q_COMPUTE];
        std::vector<int32_t> &in_ids = pool->v_plan_in;
        if (pool->group_lists.size() < (size_t)MAX_GROUP_LAYERS) pool->group_lists.resize(MAX_GROUP_LAYERS);
        std::vector<SwapList> &lists = pool->group_lists;
        for (SwapList &sl : lists) sl.n_moved = 0;
        size_t n_lists = 0;
        for (int32_t d = 0; d < next_len && L > 1 && st == PIE_OK; ++d) {
            const int32_t target = next_first + d;
            if (target >= l && target < l + pool->group_len) continue;   // fewer layers than two groups
            plan_in(pool, target, in_ids);
            if (in_ids.empty()) continue;
            st = swap_prepare(pool, PIE_Q_IN, target, in_ids.data(), (int64_t)in_ids.size(), &lists[n_lists++]);
            if (st == PIE_OK && lists[n_lists - 1].n_moved > 0) count_prefetch(pool, target < l);
        }
        const int st2 = swap_issue_group(pool, PIE_Q_IN, lists, mode, start_with);   // what was prepared must be issued
        if (st != PIE_OK) return st;
        if (st2 != PIE_OK) return st2;
    }
    // units of this layer that nobody prefetched (the very first layers of a run, a caller that skipped a layer, a
    // share the pool had no room for): fetch them now; the attention call waits for the copy
    {
        pool->v_in.clear();
        for (int32_t b : candidate_ids(pool, l))
            if (pool->table->unit(l, b).side == PIE_HOST) pool->v_in.push_back(b);
        if (!pool->v_in.empty()) {
            std::vector<int32_t> ids(pool->v_in);
            st = pool_swap(pool, PIE_Q_IN, l, ids.data(), (int64_t)ids.size(), mode);
            if (st != PIE_OK) return st;   // nothing of this layer has been enqueued
        }
    }
    // (long work items only where the library runs the layers back to back: a caller that goes layer by layer puts its own
    // kernels between two attention launches, nothing hides a launch's tail there, and the pool's chunk balances it better -
    // measured with 70 us of other work per layer on the 7B shape: 9.16 ms per step with 512-token items, 9.61 with 2048)
    st = attention_call(pool, l, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, nullptr, nullptr, n_seqs, scale,
                        k_new, v_new, dependent, defer, dependent || defer);
    if (st != PIE_OK) return st;
    pool->group_done.push_back(l);
    if ((int32_t)pool->group_done.size() >= pool->group_len) return finish_group(pool);
    return PIE_OK;
}

int pie_decode_step(pie_pool *pool, const void *q_all, void *out_all, const int32_t *block_table_dev, int32_t max_blocks_per_seq,
                    const int32_t *ctx_lens_dev, int32_t n_seqs, float scale, const void *k_new_all, const void *v_new_all,
                    int32_t mode) {
    if (!pool || !q_all || !out_all) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (pool->fifo)
        return decode_step_layers(pool, q_all, out_all, block_table_dev, max_blocks_per_seq, ctx_lens_dev, n_seqs, scale,
                                  k_new_all, v_new_all, mode);
    const int32_t L = pool->cfg.n_layers;
    const int64_t q_stride = (int64_t)n_seqs * pool->cfg.n_q_heads * pool->cfg.head_dim * 2;
    const int64_t kv_stride = (int64_t)n_seqs * pool->cfg.n_kv_heads * pool->cfg.head_dim * 2;
    int st = pie_step_begin(pool);
    if (st != PIE_OK) return st;
    for (int32_t l = 0; l < L; ++l) {
        st = decode_layer(pool, l, (const uint8_t *)q_all + l * q_stride, (uint8_t *)out_all + l * q_stride, block_table_dev,
                          max_blocks_per_seq, ctx_lens_dev, n_seqs, scale,
                          k_new_all ? (const uint8_t *)k_new_all + l * kv_stride : nullptr,
                          v_new_all ? (const uint8_t *)v_new_all + l * kv_stride : nullptr, mode, l > 0, l + 1 < L);
        if (st != PIE_OK) {
            flush_deferred_combine(pool);   // the layers already enqueued keep their results
            return st;
        }
    }
    return pie_controller_tick(pool, nullptr);
}

int pie_decode_layer(pie_pool *pool, int32_t layer, const void *q, void *out, const int32_t *block_table_dev,
                     int32_t max_blocks_per_seq, const int32_t *ctx_lens_dev, int32_t n_seqs, float scale, const void *k_new,
                     const void *v_new, int32_t mode) {
    if (!pool || !q || !out) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    if (pool->fifo) return PIE_ERR_UNSUPPORTED;  // the whole-layer protocol is driven by pie_decode_step
    if (layer < 0 || layer >= pool->cfg.n_layers) return PIE_ERR_RANGE;
    return decode_layer(pool, layer, q, out, block_table_dev, max_blocks_per_seq, ctx_lens_dev, n_seqs, scale, k_new, v_new, mode);
}

int pie_decode_step_host(pie_pool *pool, const void *q_all_host, void *out_all_host, const int32_t *block_table_host,
                         int32_t max_blocks_per_seq, const int32_t *ctx_lens_host, int32_t n_seqs, float scale,
                         const void *k_new_all_host, const void *v_new_all_host, int32_t mode) {
    if (!pool || !q_all_host || !out_all_host || !block_table_host || !ctx_lens_host) return PIE_ERR_INVALID;
    if (n_seqs <= 0 || n_seqs > pool->scratch.max_seqs || max_blocks_per_seq <= 0) return PIE_ERR_INVALID;
    if ((k_new_all_host == nullptr) != (v_new_all_host == nullptr)) return PIE_ERR_INVALID;
    if (pool->sticky != PIE_OK) return pool->sticky;
    int st = ensure_stage(pool, n_seqs, max_blocks_per_seq);
    if (st != PIE_OK) return st;
    cudaStream_t s = pool->stream[PIE_Q_COMPUTE];
    const int32_t L = pool->cfg.n_layers;
    const int64_t q_layer = (int64_t)n_seqs * pool->cfg.n_q_heads * pool->cfg.head_dim * 2;
    const int64_t kv_layer = (int64_t)n_seqs * pool->cfg.n_kv_heads * pool->cfg.head_dim * 2;
    const int64_t qb = L * q_layer, kb = L * kv_layer;
    // the host tables say which block of each sequence the append writes: kept host copies of the others stay good
    struct AppendGuard {
        pie_pool *p;
        std::vector<int32_t> saved;
        bool declared, active = false;
        ~AppendGuard() {
            if (!active) return;
            p->append_ids.swap(saved);
            p->append_declared = declared;
        }
    } guard{pool, {}, pool->append_declared};
    if (k_new_all_host && pool->table->tracks_writes()) {
        guard.saved.swap(pool->append_ids);
        guard.active = true;
        for (int32_t sq = 0; sq < n_seqs; ++sq)
            if (ctx_lens_host[sq] > 0 && ctx_lens_host[sq] <= max_blocks_per_seq * 16)
                pool->append_ids.push_back(block_table_host[(int64_t)sq * max_blocks_per_seq + (ctx_lens_host[sq] - 1) / 16]);
        pool->append_declared = true;
    }
    PIE_CUDA(cudaMemcpyAsync(pool->stage_bt, block_table_host, (size_t)n_seqs * max_blocks_per_seq * 4, cudaMemcpyHostToDevice, s));
    PIE_CUDA(cudaMemcpyAsync(pool->stage_ctx, ctx_lens_host, (size_t)n_seqs * 4, cudaMemcpyHostToDevice, s));
    if (pool->fifo) {
        // whole-layer protocol: the step is driven as a whole; inputs go up first, results come down last
        PIE_CUDA(cudaMemcpyAsync(pool->stage_q, q_all_host, (size_t)qb, cudaMemcpyHostToDevice, s));
        if (k_new_all_host) {
            PIE_CUDA(cudaMemcpyAsync(pool->stage_k, k_new_all_host, (size_t)kb, cudaMemcpyHostToDevice, s));
            PIE_CUDA(cudaMemcpyAsync(pool->stage_v, v_new_all_host, (size_t)kb, cudaMemcpyHostToDevice, s));
        }
        st = pie_decode_step(pool, pool->stage_q, pool->stage_out, pool->stage_bt, max_blocks_per_seq, pool->stage_ctx, n_seqs,
                             scale, k_new_all_host ? pool->stage_k : nullptr, k_new_all_host ? pool->stage_v : nullptr, mode);
        if (st != PIE_OK) return st;
        PIE_CUDA(cudaMemcpyAsync(out_all_host, pool->stage_out, (size_t)qb, cudaMemcpyDeviceToHost, s));
        PIE_CUDA(cudaStreamSynchronize(s));
        return check_status_word(pool);
    }
    // Pipelined by groups of layers on two streams of their own (not the swap streams: a prefetch must not queue
    // behind an upload): a group's inputs go up while the groups before it compute, its results come down while the
    // groups after it compute.  The previous call ended with a synchronisation, so the staging buffers are free.
    st = ensure_io(pool);
    if (st != PIE_OK) return st;
    const int32_t G = IO_GROUP_LAYERS, n_groups = (L + G - 1) / G;
    for (int32_t g = 0; g < n_groups; ++g) {
        const int32_t l0 = g * G, nl = std::min(G, L - l0);
        PIE_CUDA(cudaMemcpyAsync((uint8_t *)pool->stage_q + l0 * q_layer, (const uint8_t *)q_all_host + l0 * q_layer,
                                 (size_t)(nl * q_layer), cudaMemcpyHostToDevice, pool->io_stream[0]));
        if (k_new_all_host) {
            PIE_CUDA(cudaMemcpyAsync((uint8_t *)pool->stage_k + l0 * kv_layer, (const uint8_t *)k_new_all_host + l0 * kv_layer,
                                     (size_t)(nl * kv_layer), cudaMemcpyHostToDevice, pool->io_stream[0]));
            PIE_CUDA(cudaMemcpyAsync((uint8_t *)pool->stage_v + l0 * kv_layer, (const uint8_t *)v_new_all_host + l0 * kv_layer,
                                     (size_t)(nl * kv_layer), cudaMemcpyHostToDevice, pool->io_stream[0]));
        }
        // the group's arrival: the count of groups brought up so far, stored behind the group's copies; the group's first
        // attention kernel waits for it itself (a stream-level wait would cost the compute stream its chain of dependent launches)
        int64_t woff = 0;
        st = list_alloc(pool, 4, &woff);
        if (st != PIE_OK) return st;
        unsigned long long *w = reinterpret_cast<unsigned long long *>(pool->list_host + woff);
        *w = ++pool->io_groups_up;
        PIE_CUDA(cudaMemcpyAsync(pool->io_arrive_dev, w, 8, cudaMemcpyHostToDevice, pool->io_stream[0]));
        st = list_commit(pool, woff, 4, pool->io_stream[0]);
        if (st != PIE_OK) return st;
    }
    const unsigned long long groups_before = pool->io_groups_up - (unsigned long long)n_groups;
    st = pie_step_begin(pool);
    if (st != PIE_OK) return st;
    int32_t pending_group = -1;   // a group whose layers are enqueued and whose results wait for the next layer's kernel
    auto download = [&](int32_t g, bool by_value) -> int {
        const int32_t l0 = g * G, nl = std::min(G, L - l0);
        int rc = PIE_OK;
        if (by_value && pool->wait_value64 && pool->recorded[PIE_Q_COMPUTE] == pool->last_attn_ticket) {
            // the kernel of the layer after the group has completed -> so has the group's last combine kernel before it
            if (pool->wait_value64((CUstream)pool->io_stream[1], (CUdeviceptr)(uintptr_t)pool->done_dev, (cuuint64_t)pool->last_attn_ticket,
                                   CU_STREAM_WAIT_VALUE_GEQ) != CUDA_SUCCESS)
                rc = PIE_ERR_CUDA;
        } else {
            cudaEvent_t ev = nullptr;
            rc = push_mark(pool, &ev);
            if (rc == PIE_OK && cudaStreamWaitEvent(pool->io_stream[1], ev, 0) != cudaSuccess) rc = PIE_ERR_CUDA;
        }
        if (rc != PIE_OK) return rc;
        PIE_CUDA(cudaMemcpyAsync((uint8_t *)out_all_host + l0 * q_layer, (const uint8_t *)pool->stage_out + l0 * q_layer,
                                 (size_t)(nl * q_layer), cudaMemcpyDeviceToHost, pool->io_stream[1]));
        return PIE_OK;
    };
    for (int32_t l = 0; l < L; ++l) {
        pool->inputs_need = l % G == 0 ? groups_before + (unsigned long long)(l / G) + 1 : 0;
        st = decode_layer(pool, l, (const uint8_t *)pool->stage_q + l * q_layer, (uint8_t *)pool->stage_out + l * q_layer,
                          pool->stage_bt, max_blocks_per_seq, pool->stage_ctx, n_seqs, scale,
                          k_new_all_host ? (const uint8_t *)pool->stage_k + l * kv_layer : nullptr,
                          k_new_all_host ? (const uint8_t *)pool->stage_v + l * kv_layer : nullptr, mode, l > 0, l + 1 < L);
        pool->inputs_need = 0;
        if (st != PIE_OK) {
            flush_deferred_combine(pool);
            break;
        }
        if (pending_group >= 0) {   // the group before this layer: its results come down once this layer's kernel has run
            st = download(pending_group, true);
            pending_group = -1;
            if (st != PIE_OK) break;
        }
        if ((l + 1) % G == 0 || l + 1 == L) pending_group = l / G;
    }
    if (st == PIE_OK && pending_group >= 0) st = download(pending_group, false);   // the last group: behind a mark
    // whatever happened, nothing of this call may still be in flight when it returns (the caller owns the host buffers)
    cudaError_t e1 = cudaStreamSynchronize(pool->io_stream[0]);
    cudaError_t e2 = cudaStreamSynchronize(s);
    cudaError_t e3 = cudaStreamSynchronize(pool->io_stream[1]);
    if (st != PIE_OK) return st;
    if (e1 != cudaSuccess || e2 != cudaSuccess || e3 != cudaSuccess) {
        g_last_cuda_error = (int)(e1 != cudaSuccess ? e1 : e2 != cudaSuccess ? e2 : e3);
        pool->sticky = PIE_ERR_CUDA;
        return PIE_ERR_CUDA;
    }
    st = pie_controller_tick(pool, nullptr);
    if (st != PIE_OK) return st;
    return check_status_word(pool);
}

int pie_probe_link(int64_t bytes, int32_t dir, int32_t reps, double *gbps) {
    if (bytes <= 0 || dir < 0 || dir > 2 || reps <= 0 || !gbps) return PIE_ERR_INVALID;
    void *h[2] = {nullptr, nullptr}, *d[2] = {nullptr, nullptr};
    cudaStream_t s[2] = {nullptr, nullptr};
    cudaEvent_t e0 = nullptr, e1[2] = {nullptr, nullptr};
    int rc = PIE_OK;
    double best = 0;
    auto cleanup = [&]() {
        for (int i = 0; i < 2; ++i) {
            if (h[i]) cudaFreeHost(h[i]);
            if (d[i]) cudaFree(d[i]);
            if (s[i]) cudaStreamDestroy(s[i]);
            if (e1[i]) cudaEventDestroy(e1[i]);
        }
        if (e0) cudaEventDestroy(e0);
    };
#define PROBE(call) do { cudaError_t e__ = (call); if (e__ != cudaSuccess) { g_last_cuda_error = (int)e__; cleanup(); return PIE_ERR_CUDA; } } while (0)
    const int n = dir == 2 ? 2 : 1;
    for (int i = 0; i < n; ++i) {
        PROBE(cudaHostAlloc(&h[i], (size_t)bytes, cudaHostAllocDefault));
        std::memset(h[i], 1, (size_t)bytes);
        PROBE(cudaMalloc(&d[i], (size_t)bytes));
        PROBE(cudaStreamCreateWithFlags(&s[i], cudaStreamNonBlocking));
        PROBE(cudaEventCreate(&e1[i]));
    }
    PROBE(cudaEventCreate(&e0));
    for (int r = 0; r < reps + 1; ++r) {  // first repetition is a warm-up
        PROBE(cudaEventRecord(e0, s[0]));
        if (n == 2) PROBE(cudaStreamWaitEvent(s[1], e0, 0));
        for (int i = 0; i < n; ++i) {
            const bool h2d = dir == PIE_H2D || (dir == 2 && i == 0);
            if (h2d) PROBE(cudaMemcpyAsync(d[i], h[i], (size_t)bytes, cudaMemcpyHostToDevice, s[i]));
            else PROBE(cudaMemcpyAsync(h[i], d[i], (size_t)bytes, cudaMemcpyDeviceToHost, s[i]));
            PROBE(cudaEventRecord(e1[i], s[i]));
        }
        float worst = 0;
        for (int i = 0; i < n; ++i) {
            PROBE(cudaEventSynchronize(e1[i]));
            float ms = 0;
            PROBE(cudaEventElapsedTime(&ms, e0, e1[i]));
            worst = std::max(worst, ms);
        }
        if (r > 0 && worst > 0) best = std::max(best, (double)bytes / (worst * 1e-3) / 1e9);
    }
#undef PROBE
    cleanup();
    *gbps = best;
    return rc;
}

int pie_probe_hbm(int64_t bytes, int32_t reps, double *gbps) {
    if (bytes <= 0 || reps <= 0 || !gbps) return PIE_ERR_INVALID;
    void *a = nullptr, *b = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    auto cleanup = [&]() {
        cudaFree(a);
        cudaFree(b);
        if (e0) cudaEventDestroy(e0);
        if (e1) cudaEventDestroy(e1);
    };
#define PROBE(call) do { cudaError_t e__ = (call); if (e__ != cudaSuccess) { g_last_cuda_error = (int)e__; cleanup(); return PIE_ERR_CUDA; } } while (0)
    PROBE(cudaMalloc(&a, (size_t)bytes));
    PROBE(cudaMalloc(&b, (size_t)bytes));
    PROBE(cudaMemset(a, 1, (size_t)bytes));
    PROBE(cudaEventCreate(&e0));
    PROBE(cudaEventCreate(&e1));
    double best = 0;
    for (int r = 0; r < reps + 1; ++r) {
        PROBE(cudaEventRecord(e0, 0));
        PROBE(cudaMemcpyAsync(b, a, (size_t)bytes, cudaMemcpyDeviceToDevice, 0));
        PROBE(cudaEventRecord(e1, 0));
        PROBE(cudaEventSynchronize(e1));
        float ms = 0;
        PROBE(cudaEventElapsedTime(&ms, e0, e1));
        if (r > 0 && ms > 0) best = std::max(best, 2.0 * (double)bytes / (ms * 1e-3) / 1e9);
    }
#undef PROBE
    cleanup();
    *gbps = best;
    return PIE_OK;
}

}  // extern "C"
