// Host-side mapping table, slot pools, whole-layer protocol scheduler and controller rule.
// Pure C++ (no CUDA): pie_pool drives it, and it is exported through the C ABI for CPU tests.
#pragma once
#include <algorithm>
#include <cstdint>
#include <deque>
#include <map>
#include <vector>

#include "../../include/pie.h"

namespace pie {

struct SlotTag {
    int32_t queue;
    int64_t ticket;
};

// Free slots of one pool.  `ready` holds slots that are free for certain, as runs of consecutive numbers; `pending`
// is a queue of slots released by a copy that may not have finished: they can be handed out, but the receiver must
// wait for the tag's ticket.  Hand-out rule (shared with the oracle, so that the two can be compared slot by slot):
// a request for n >= 2 slots looks, in ascending order, for the first ready run that has n slots at or after the
// cursor and takes the first n of those; failing that (and for a single slot, which leaves the cursor alone), the first
// n of the lowest ready run that has at least n; failing that, whole runs, longest first (lowest first among equals),
// until it is served; the cursor then stands behind the slots taken last.  What ready cannot give comes from the front
// of pending.  The slots of swap lists are released in about the order they were taken, so the hand-out walks round the
// pool's spare part like a ring: lists land in consecutive slots, and consecutive lists beside each other, whatever
// their sizes were before - which is what lets a few large copies move them.  (Taking the lowest run that fits, the
// rule before this one, serves a steady ratio as well but splinters the spare part once the lists grow and shrink by a
// few blocks at a time: after a ramp of the adaptive controller a list of 20 blocks came in three runs.)  Allocations,
// which live long - single slots, and the pool's layer-by-layer requests for several blocks at once - fill the lowest
// runs that fit and stay out of the ring's way.
class SlotPool {
  public:
    explicit SlotPool(int64_t n);
    void settle(const int64_t *done);
    int64_t available() const { return n_ready_ + (int64_t)pending_.size(); }
    // n slots into slots[0..n), their tags into tags[0..n); the caller has checked available() >= n
    // lists = false: an allocation (long-lived): the cursor is neither used nor moved
    void take_n(int64_t n, int32_t *slots, SlotTag *tags, bool lists = true);
    int32_t take(SlotTag *tag) {
        int32_t s;
        take_n(1, &s, tag);
        return s;
    }
    void release(int32_t slot, int32_t queue, int64_t ticket);

  private:
    struct Pending {
        int32_t slot;
        int32_t queue;
        int64_t ticket;
    };
    void add_ready(int32_t slot);
    void add_ready_run(int32_t start, int32_t len);
    std::map<int32_t, int32_t> runs_;  // start -> length of a run of ready slots
    int64_t n_ready_ = 0;
    int32_t cursor_ = 0;  // behind the slots that the last request of two or more took from ready
    std::deque<Pending> pending_;
};

struct Unit {
    uint8_t side = PIE_FREE;  // PIE_FREE / PIE_GPU / PIE_HOST: where the unit is or is heading
    uint8_t last_q = PIE_Q_NONE;
    uint8_t home_host = 0;  // belongs to the host-resident set between uses
    uint8_t dirty = 0;      // written on the GPU since its host copy was taken (matters while a host slot is kept)
    int32_t gpu_slot = -1;
    int32_t host_slot = -1;
    int64_t last_t = 0;
    uint32_t t_stamp = 0;  // the table's timestamp column (Section 3.2)
};

class Table {
  public:
    Table(int32_t n_layers, int32_t n_logical, int64_t n_gpu_slots, int64_t n_host_slots);

    int alloc(int32_t block, bool on_host);
    // n blocks at once, slots handed out layer by layer so that each layer's units sit in consecutive slots
    int alloc_bulk(const int32_t *blocks, int64_t n, const uint8_t *on_host);
    int free_block(int32_t block);
    // elide (optional, capacity n): 1 where the pair needs no bytes moved (a kept, unwritten host copy)
    int swap(int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int32_t *moved,
             int32_t *src, int32_t *dst, int64_t *n_moved, int64_t *waits, uint8_t *elide = nullptr);
    // Variant beyond the paper (Section 3.2 gives the CPU region up after a swap-in): a unit that comes in keeps
    // its host slot, and going out again copies nothing unless it was marked written meanwhile.
    void set_retain(bool on) { retain_ = on; }
    bool retain() const { return retain_; }
    // GPU-resident units that hold a kept host copy: while there are any, whoever writes a unit has to mark it dirty,
    // whether or not the switch is still on (switching it off takes effect unit by unit at the next swap-in)
    int64_t kept_copies() const { return n_kept_; }
    bool tracks_writes() const { return retain_ || n_kept_ > 0; }
    int mark_dirty(int32_t layer, const int32_t *ids, int64_t n);
    int drop_host_copy(int32_t layer, int32_t block);  // a GPU-resident unit gives its kept host slot up
    void mark_layer_dirty(int32_t layer);
    int attention(int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int64_t *waits);
    int confirm(int32_t queue, int64_t ticket);

    // Run-time resize of the per-layer size (Section 4.1).  NB is the physical width; ids below capacity()
    // are visible.  Growing: new ids become allocatable once every layer has gone through a swap pass;
    // shrinking: ids at or above the new size stop being handed out at once and the size takes effect
    // once every layer has passed (blocks still in use up there stay accessible until freed).
    int init_capacity(int32_t size);  // before anything is allocated
    int resize_begin(int32_t new_size);
    bool layer_pass(int32_t layer);  // true when this call completed a resize
    int32_t capacity() const { return capacity_; }
    int32_t resize_target() const { return target_; }  // -1: none in progress
    int32_t layers_moved() const { return n_moved_; }
    int32_t alloc_limit() const { return target_ < 0 ? capacity_ : std::min(capacity_, target_); }
    int state(int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot, int32_t *host_slot);

    bool in_flight(const Unit &u) const { return u.last_q != PIE_Q_NONE && u.last_t > done_[u.last_q]; }
    Unit &unit(int32_t layer, int32_t block) { return units_[(int64_t)layer * NB + block]; }
    bool allocated(int32_t block) const { return allocated_[block] != 0; }
    int64_t gpu_available() { settle(); return gpu_.available(); }
    int64_t host_available() { settle(); return host_.available(); }
    int64_t issued(int q) const { return issued_[q]; }
    int64_t done(int q) const { return done_[q]; }
    int32_t n_allocated() const { return n_allocated_; }
    // a slot goes to `pending` only with a ticket that is still open, so nothing can move while `done_` stands still
    void settle() {
        if (settled_[1] == done_[1] && settled_[2] == done_[2] && settled_[3] == done_[3]) return;
        gpu_.settle(done_);
        host_.settle(done_);
        for (int q = 0; q < 4; ++q) settled_[q] = done_[q];
    }

    const int32_t L, NB;

  private:
    int check_ids(int32_t layer, const int32_t *ids, int64_t n);
    SlotPool gpu_, host_;
    std::vector<Unit> units_;
    std::vector<uint8_t> allocated_;
    std::vector<uint32_t> seen_;  // duplicate detection: seen_[block] == stamp
    uint32_t seen_stamp_ = 0;
    std::vector<int64_t> last_compute_;      // per layer
    std::vector<int64_t> layer_wait_;        // per layer x 4 queues: newest open ticket among its units
    int64_t issued_[4] = {0, 0, 0, 0};
    int64_t done_[4] = {0, 0, 0, 0};
    int64_t settled_[4] = {0, 0, 0, 0};  // done_ as of the last settle()
    uint32_t clock_ = 0;
    int32_t n_allocated_ = 0;
    int32_t capacity_, target_ = -1, n_moved_ = 0;
    bool retain_ = false;
    int64_t n_kept_ = 0;
    std::vector<uint8_t> moved_;  // per layer
    std::vector<int32_t> take_slots_;  // scratch of swap() / alloc_bulk()
    std::vector<SlotTag> take_tags_;
};

// Whole-layer protocol of Section 3.3.
class Fifo {
  public:
    Fifo(int32_t n, int32_t gpu_regions, int32_t cpu_regions, const uint8_t *on_cpu);
    int complete(int32_t dir);
    int layer_start(int32_t k, int32_t *start_out, int32_t *start_in);
    int location(int32_t layer) const;
    int64_t in_starts() const { return in_starts_; }     // swap-ins started so far
    int64_t violations() const { return violations_; }   // ... of which for a layer of the next token

  private:
    int64_t in_starts_ = 0, violations_ = 0;
    int32_t n_, gpu_regions_, cpu_regions_;
    std::vector<uint8_t> loc_;  // 0 GPU, 1 CPU, 2 to CPU, 3 to GPU
    int32_t out_layer_ = -1, in_layer_ = -1;
};

}  // namespace pie
