// Mapping table with stream-ordered two-phase updates (Section 3.2), the whole-layer swap protocol
// (Section 3.3) and the controller's decision rule (Section 3.4.2).  Host only.
#include "pie_table.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <new>

namespace pie {

// ------------------------------------------------------------------------------------ SlotPool
SlotPool::SlotPool(int64_t n) {
    if (n > 0) runs_[0] = (int32_t)n;
    n_ready_ = n;
}

void SlotPool::add_ready_run(int32_t start, int32_t len) {
    // one map operation per run of consecutive slots: joined to the run before it and / or the run after it
    auto next = runs_.lower_bound(start);
    int32_t s = start, l = len;
    if (next != runs_.begin()) {
        auto prev = std::prev(next);
        if (prev->first + prev->second == start) {  // extends the run before it
            s = prev->first;
            l += prev->second;
            runs_.erase(prev);
        }
    }
    if (next != runs_.end() && next->first == start + len) {  // closes the gap to the run after it
        l += next->second;
        runs_.erase(next);
    }
    runs_[s] = l;
    n_ready_ += len;
}

void SlotPool::add_ready(int32_t slot) { add_ready_run(slot, 1); }

void SlotPool::settle(const int64_t *done) {
    if (pending_.empty()) return;
    // swap lists release their slots in runs: confirmed neighbours in the queue that are neighbours in the pool go in as one
    size_t keep = 0;
    int32_t run_start = 0, run_len = 0;
    for (size_t i = 0; i < pending_.size(); ++i) {
        const Pending p = pending_[i];
        if (p.ticket <= done[p.queue]) {
            if (run_len > 0 && p.slot == run_start + run_len) {
                ++run_len;
            } else {
                if (run_len > 0) add_ready_run(run_start, run_len);
                run_start = p.slot;
                run_len = 1;
            }
        } else {
            pending_[keep++] = p;
        }
    }
    if (run_len > 0) add_ready_run(run_start, run_len);
    pending_.resize(keep);
}

void SlotPool::take_n(int64_t n, int32_t *slots, SlotTag *tags, bool lists) {
    int64_t k = 0;
    const bool rove = lists && n >= 2;
    while (k < n && !runs_.empty()) {
        const int64_t want = n - k;
        auto pick = runs_.end();
        int32_t from = 0;
        if (rove)  // the first run that has `want` slots at or after the cursor
            for (auto it = runs_.begin(); it != runs_.end(); ++it) {
                const int32_t a = std::max(it->first, cursor_);
                if ((int64_t)it->first + it->second - a >= want) {
                    pick = it;
                    from = a;
                    break;
                }
            }
        if (pick == runs_.end()) {
            auto longest = runs_.begin();
            for (auto it = runs_.begin(); it != runs_.end(); ++it) {
                if (it->second >= want) {
                    pick = it;  // the lowest run that serves the rest of the request
                    break;
                }
                if (it->second > longest->second) longest = it;
            }
            if (pick == runs_.end()) pick = longest;
            from = pick->first;
        }
        const int32_t start = pick->first, len = pick->second;
        const int32_t m = (int32_t)std::min<int64_t>(want, (int64_t)start + len - from);
        for (int32_t i = 0; i < m; ++i) {
            slots[k] = from + i;
            tags[k].queue = PIE_Q_NONE;
            tags[k].ticket = 0;
            ++k;
        }
        runs_.erase(pick);
        if (from > start) runs_[start] = from - start;
        if (from + m < start + len) runs_[from + m] = start + len - (from + m);
        n_ready_ -= m;
        if (rove) cursor_ = from + m;
    }
    while (k < n) {
        Pending p = pending_.front();
        pending_.pop_front();
        slots[k] = p.slot;
        tags[k].queue = p.queue;
        tags[k].ticket = p.ticket;
        ++k;
    }
}

void SlotPool::release(int32_t slot, int32_t queue, int64_t ticket) {
    if (queue == PIE_Q_NONE) add_ready(slot);
    else pending_.push_back({slot, queue, ticket});
}

// --------------------------------------------------------------------------------------- Table
Table::Table(int32_t n_layers, int32_t n_logical, int64_t n_gpu_slots, int64_t n_host_slots)
    : L(n_layers), NB(n_logical), gpu_(n_gpu_slots), host_(n_host_slots),
      units_((size_t)n_layers * (size_t)n_logical), allocated_((size_t)n_logical, 0), seen_((size_t)n_logical, 0),
      last_compute_((size_t)n_layers, 0), layer_wait_((size_t)n_layers * 4, 0), capacity_(n_logical),
      moved_((size_t)n_layers, 0) {}

int Table::init_capacity(int32_t size) {
    if (size <= 0 || size > NB) return PIE_ERR_RANGE;
    if (n_allocated_ != 0 || target_ >= 0) return PIE_ERR_BUSY;
    capacity_ = size;
    return PIE_OK;
}

int Table::resize_begin(int32_t new_size) {
    if (new_size <= 0 || new_size > NB) return PIE_ERR_RANGE;
    if (target_ >= 0) return PIE_ERR_BUSY;
    if (new_size != capacity_) {
        target_ = new_size;
        n_moved_ = 0;
        std::fill(moved_.begin(), moved_.end(), (uint8_t)0);
    }
    return PIE_OK;
}

bool Table::layer_pass(int32_t layer) {
    if (target_ < 0 || layer < 0 || layer >= L) return false;
    if (!moved_[(size_t)layer]) {
        moved_[(size_t)layer] = 1;
        ++n_moved_;
    }
    if (n_moved_ < L) return false;
    capacity_ = target_;
    target_ = -1;
    n_moved_ = 0;
    return true;
}

int Table::alloc(int32_t block, bool on_host) {
    if (block < 0 || block >= NB) return PIE_ERR_RANGE;
    if (block >= alloc_limit()) return PIE_ERR_NOMEM;  // beyond the size visible now
    if (allocated_[block]) return PIE_ERR_INVALID;
    settle();
    int64_t n_gpu = on_host ? 0 : std::min<int64_t>(L, gpu_.available());
    if (L - n_gpu > host_.available()) return PIE_ERR_NOMEM;
    for (int32_t l = 0; l < L; ++l) {
        Unit &u = unit(l, block);
        SlotTag tag;
        if (l < n_gpu) {
            u.gpu_slot = gpu_.take(&tag);
            u.host_slot = -1;
            u.side = PIE_GPU;
            u.home_host = 0;
        } else {
            u.host_slot = host_.take(&tag);
            u.gpu_slot = -1;
            u.side = PIE_HOST;
            u.home_host = 1;
        }
        // a recycled slot whose ticket is open makes the new unit "in flight" on that ticket
        u.last_q = (uint8_t)tag.queue;
        u.last_t = tag.ticket;
        if (tag.queue != PIE_Q_NONE) {
            int64_t &w = layer_wait_[(size_t)l * 4 + tag.queue];
            w = std::max(w, tag.ticket);
        }
        u.t_stamp = clock_;
    }
    allocated_[block] = 1;
    ++n_allocated_;
    return PIE_OK;
}

int Table::alloc_bulk(const int32_t *blocks, int64_t n, const uint8_t *on_host) {
    settle();
    for (int64_t i = 0; i < n; ++i) {
        if (blocks[i] < 0 || blocks[i] >= NB) return PIE_ERR_RANGE;
        if (blocks[i] >= alloc_limit()) return PIE_ERR_NOMEM;
        if (allocated_[blocks[i]]) return PIE_ERR_INVALID;
    }
    // budget: a block that is not forced to the host takes GPU slots for its first layers while any are left
    std::vector<int32_t> n_gpu((size_t)n, 0);
    int64_t gpu_left = gpu_.available(), need_host = 0;
    for (int64_t i = 0; i < n; ++i) {
        n_gpu[(size_t)i] = on_host && on_host[i] ? 0 : (int32_t)std::min<int64_t>(L, gpu_left);
        gpu_left -= n_gpu[(size_t)i];
        need_host += L - n_gpu[(size_t)i];
    }
    if (need_host > host_.available()) return PIE_ERR_NOMEM;
    std::vector<int32_t> host_slots;
    std::vector<SlotTag> host_tags;
    for (int32_t l = 0; l < L; ++l) {
        // one request per layer and side: a layer's units sit in consecutive slots where the pools allow
        int64_t want_gpu = 0;
        for (int64_t i = 0; i < n; ++i) want_gpu += l < n_gpu[(size_t)i];
        take_slots_.resize((size_t)want_gpu);
        take_tags_.resize((size_t)want_gpu);
        host_slots.resize((size_t)(n - want_gpu));
        host_tags.resize((size_t)(n - want_gpu));
        // (allocations live long: they fill the lowest runs that fit and leave the swap lists' cursor alone)
        if (want_gpu > 0) gpu_.take_n(want_gpu, take_slots_.data(), take_tags_.data(), false);
        if (n - want_gpu > 0) host_.take_n(n - want_gpu, host_slots.data(), host_tags.data(), false);
        int64_t ig = 0, ih = 0;
        for (int64_t i = 0; i < n; ++i) {
            Unit &u = unit(l, blocks[i]);
            SlotTag tag;
            if (l < n_gpu[(size_t)i]) {
                tag = take_tags_[(size_t)ig];
                u.gpu_slot = take_slots_[(size_t)ig++];
                u.host_slot = -1;
                u.side = PIE_GPU;
                u.home_host = 0;
            } else {
                tag = host_tags[(size_t)ih];
                u.host_slot = host_slots[(size_t)ih++];
                u.gpu_slot = -1;
                u.side = PIE_HOST;
                u.home_host = 1;
            }
            u.last_q = (uint8_t)tag.queue;
            u.last_t = tag.ticket;
            if (tag.queue != PIE_Q_NONE) {
                int64_t &w = layer_wait_[(size_t)l * 4 + tag.queue];
                w = std::max(w, tag.ticket);
            }
            u.t_stamp = clock_;
        }
    }
    for (int64_t i = 0; i < n; ++i) allocated_[blocks[i]] = 1;
    n_allocated_ += (int32_t)n;
    return PIE_OK;
}

int Table::free_block(int32_t block) {
    if (block < 0 || block >= NB) return PIE_ERR_RANGE;
    if (!allocated_[block]) return PIE_ERR_INVALID;
    settle();
    for (int32_t l = 0; l < L; ++l)
        if (in_flight(unit(l, block))) return PIE_ERR_BUSY;
    for (int32_t l = 0; l < L; ++l) {
        Unit &u = unit(l, block);
        if (u.side == PIE_GPU) {
            // an attention call issued earlier may still be reading the slot
            int64_t ct = issued_[PIE_Q_COMPUTE];
            gpu_.release(u.gpu_slot, ct > done_[PIE_Q_COMPUTE] ? PIE_Q_COMPUTE : PIE_Q_NONE, ct);
            if (u.host_slot >= 0) {  // a kept host copy goes with the unit
                host_.release(u.host_slot, PIE_Q_NONE, 0);
                --n_kept_;
            }
        } else {
            host_.release(u.host_slot, PIE_Q_NONE, 0);
        }
        u = Unit();
    }
    allocated_[block] = 0;
    --n_allocated_;
    return PIE_OK;
}

int Table::check_ids(int32_t layer, const int32_t *ids, int64_t n) {
    if (layer < 0 || layer >= L) return PIE_ERR_RANGE;
    if (n < 0 || (n > 0 && !ids)) return PIE_ERR_INVALID;
    if (++seen_stamp_ == 0) {  // wrapped: clear
        std::fill(seen_.begin(), seen_.end(), 0u);
        seen_stamp_ = 1;
    }
    for (int64_t i = 0; i < n; ++i) {
        int32_t b = ids[i];
        if (b < 0 || b >= NB) return PIE_ERR_RANGE;
        if (seen_[b] == seen_stamp_ || !allocated_[b]) return PIE_ERR_INVALID;
        seen_[b] = seen_stamp_;
    }
    return PIE_OK;
}

int Table::drop_host_copy(int32_t layer, int32_t block) {
    if (layer < 0 || layer >= L || block < 0 || block >= NB) return PIE_ERR_RANGE;
    if (!allocated_[block]) return PIE_ERR_INVALID;
    settle();
    Unit &u = unit(layer, block);
    if (u.side == PIE_GPU && u.host_slot >= 0) {
        // the copy that is bringing the unit in may still be reading the slot: its next owner waits for that copy
        if (in_flight(u)) host_.release(u.host_slot, u.last_q, u.last_t);
        else host_.release(u.host_slot, PIE_Q_NONE, 0);
        u.host_slot = -1;
        --n_kept_;
    }
    return PIE_OK;
}

int Table::mark_dirty(int32_t layer, const int32_t *ids, int64_t n) {
    int st = check_ids(layer, ids, n);
    if (st != PIE_OK) return st;
    for (int64_t i = 0; i < n; ++i) unit(layer, ids[i]).dirty = 1;
    return PIE_OK;
}

void Table::mark_layer_dirty(int32_t layer) {
    for (int32_t b = 0; b < NB; ++b)
        if (allocated_[b]) unit(layer, b).dirty = 1;
}

int Table::swap(int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int32_t *moved,
                int32_t *src, int32_t *dst, int64_t *n_moved, int64_t *waits, uint8_t *elide) {
    if (queue != PIE_Q_IN && queue != PIE_Q_OUT) return PIE_ERR_INVALID;
    int st = check_ids(layer, ids, n);
    if (st != PIE_OK) return st;
    settle();
    const uint8_t want = queue == PIE_Q_OUT ? PIE_HOST : PIE_GPU;
    // a unit that kept its host slot goes back into it: only the others need a new one
    int64_t movers = 0, need = 0;
    for (int64_t i = 0; i < n; ++i) {
        const Unit &u = unit(layer, ids[i]);
        if (u.side == want) continue;
        ++movers;
        if (queue == PIE_Q_IN || u.host_slot < 0) ++need;
    }
    SlotPool &dst_pool = queue == PIE_Q_OUT ? host_ : gpu_;
    SlotPool &src_pool = queue == PIE_Q_OUT ? gpu_ : host_;
    if (need > dst_pool.available()) return PIE_ERR_NOMEM;
    layer_pass(layer);
    waits[0] = waits[1] = waits[2] = waits[3] = 0;
    *n_moved = 0;
    *ticket = 0;
    if (movers == 0) return PIE_OK;
    const int64_t tk = ++issued_[queue];
    ++clock_;
    // the new slots of the whole list in one request, so that they are consecutive where the pool allows
    take_slots_.resize((size_t)need);
    take_tags_.resize((size_t)need);
    if (need > 0) dst_pool.take_n(need, take_slots_.data(), take_tags_.data());
    int64_t k = 0, taken = 0;
    for (int64_t i = 0; i < n; ++i) {
        Unit &u = unit(layer, ids[i]);
        if (u.side == want) continue;
        const bool kept = queue == PIE_Q_OUT && u.host_slot >= 0;
        int32_t d = u.host_slot;
        if (!kept) {
            const SlotTag tag = take_tags_[(size_t)taken];
            d = take_slots_[(size_t)taken++];
            if (tag.queue != PIE_Q_NONE) waits[tag.queue] = std::max(waits[tag.queue], tag.ticket);
        }
        // the copy that is still bringing the unit to where it is now
        if (in_flight(u)) waits[u.last_q] = std::max(waits[u.last_q], u.last_t);
        int32_t s;
        bool skip = false;
        if (queue == PIE_Q_OUT) {
            s = u.gpu_slot;
            skip = kept && !u.dirty;  // the kept copy is still good unless the unit was written
            if (kept) --n_kept_;
            u.host_slot = d;
            u.gpu_slot = -1;
            u.dirty = 0;
            src_pool.release(s, queue, tk);
        } else {
            s = u.host_slot;
            u.gpu_slot = d;
            if (!retain_) {
                u.host_slot = -1;
                src_pool.release(s, queue, tk);
            } else {
                ++n_kept_;
            }
            // with retain_ the host slot stays the unit's, and a dirty mark made before the unit came in survives
        }
        if (elide) elide[k] = skip ? 1 : 0;
        u.side = want;
        u.last_q = (uint8_t)queue;
        u.last_t = tk;
        u.t_stamp = clock_;
        moved[k] = ids[i];
        src[k] = s;
        dst[k] = d;
        ++k;
    }
    if (queue == PIE_Q_OUT && last_compute_[layer] > done_[PIE_Q_COMPUTE])
        // the layer's attention call also appends the new token: copy out only after it
        waits[PIE_Q_COMPUTE] = std::max(waits[PIE_Q_COMPUTE], last_compute_[layer]);
    if (queue == PIE_Q_IN) layer_wait_[(size_t)layer * 4 + PIE_Q_IN] = tk;
    waits[queue] = 0;  // same queue: ordered anyway
    for (int q = 1; q < 4; ++q)
        if (waits[q] <= done_[q]) waits[q] = 0;
    *n_moved = k;
    *ticket = tk;
    return PIE_OK;
}

int Table::attention(int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int64_t *waits) {
    int st = check_ids(layer, ids, ids ? n : 0);
    if (st != PIE_OK) return st;
    settle();
    waits[0] = waits[1] = waits[2] = waits[3] = 0;
    if (ids) {
        for (int64_t i = 0; i < n; ++i)
            if (unit(layer, ids[i]).side != PIE_GPU) return PIE_ERR_NOT_RESIDENT;
        for (int64_t i = 0; i < n; ++i) {
            const Unit &u = unit(layer, ids[i]);
            if (in_flight(u)) waits[u.last_q] = std::max(waits[u.last_q], u.last_t);
        }
    } else {
        for (int q = 1; q < 4; ++q) waits[q] = layer_wait_[(size_t)layer * 4 + q];
    }
    waits[PIE_Q_COMPUTE] = 0;
    for (int q = 1; q < 4; ++q)
        if (waits[q] <= done_[q]) waits[q] = 0;
    *ticket = ++issued_[PIE_Q_COMPUTE];
    last_compute_[layer] = *ticket;
    return PIE_OK;
}

int Table::confirm(int32_t queue, int64_t ticket) {
    if (queue < 1 || queue > 3) return PIE_ERR_INVALID;
    if (ticket > issued_[queue]) return PIE_ERR_RANGE;
    if (ticket > done_[queue]) done_[queue] = ticket;
    settle();
    return PIE_OK;
}

int Table::state(int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot, int32_t *host_slot) {
    if (layer < 0 || layer >= L || block < 0 || block >= NB) return PIE_ERR_RANGE;
    const Unit &u = unit(layer, block);
    int32_t s = u.side;
    if (s != PIE_FREE && in_flight(u)) s = u.side == PIE_GPU ? PIE_TO_GPU : PIE_TO_HOST;
    if (state) *state = s;
    if (gpu_slot) *gpu_slot = u.gpu_slot;
    if (host_slot) *host_slot = u.host_slot;
    return PIE_OK;
}

// ---------------------------------------------------------------------------------------- Fifo
Fifo::Fifo(int32_t n, int32_t gpu_regions, int32_t cpu_regions, const uint8_t *on_cpu)
    : n_(n), gpu_regions_(gpu_regions), cpu_regions_(cpu_regions), loc_((size_t)n, 0) {
    for (int32_t l = 0; l < n; ++l) loc_[l] = on_cpu && on_cpu[l] ? 1 : 0;
}

int Fifo::complete(int32_t dir) {
    if (dir == PIE_Q_OUT) {
        if (out_layer_ < 0) return PIE_ERR_INVALID;
        loc_[out_layer_] = 1;  // now on the CPU: its GPU region is free
        out_layer_ = -1;
    } else if (dir == PIE_Q_IN) {
        if (in_layer_ < 0) return PIE_ERR_INVALID;
        loc_[in_layer_] = 0;  // usable on the GPU: its CPU region is free
        in_layer_ = -1;
    } else {
        return PIE_ERR_INVALID;
    }
    return PIE_OK;
}

int Fifo::location(int32_t layer) const {
    if (layer < 0 || layer >= n_) return PIE_ERR_RANGE;
    return loc_[layer];
}

int Fifo::layer_start(int32_t k, int32_t *start_out, int32_t *start_in) {
    if (k < 0 || k >= n_ || !start_out || !start_in) return PIE_ERR_INVALID;
    *start_out = *start_in = -1;
    auto dist = [&](int32_t l) { return ((l - k) % n_ + n_) % n_; };  // compute-steps until l is needed
    int32_t gpu_used = 0, cpu_used = 0;
    for (int32_t l = 0; l < n_; ++l) {
        gpu_used += loc_[l] != 1;
        cpu_used += loc_[l] != 0;
    }
    if (out_layer_ < 0 && cpu_used < cpu_regions_) {
        // coldest GPU layer other than k: next use farthest away (the layer that just finished)
        int32_t victim = -1;
        for (int32_t l = 0; l < n_; ++l)
            if (loc_[l] == 0 && l != k && (victim < 0 || dist(l) > dist(victim))) victim = l;
        bool hotter_on_cpu = false;
        if (victim >= 0)
            for (int32_t l = 0; l < n_; ++l)
                if (loc_[l] == 1 && dist(l) < dist(victim)) hotter_on_cpu = true;
        if (hotter_on_cpu) {  // otherwise every CPU layer is colder: no swap-out
            loc_[victim] = 2;
            out_layer_ = victim;
            *start_out = victim;
            ++cpu_used;
        }
    }
    if (in_layer_ < 0 && gpu_used < gpu_regions_) {
        int32_t hot = -1;
        for (int32_t l = 0; l < n_; ++l)
            if (loc_[l] == 1 && (hot < 0 || dist(l) < dist(hot))) hot = l;
        if (hot >= 0) {
            loc_[hot] = 3;
            in_layer_ = hot;
            *start_in = hot;
            // the token being computed still needs layers k .. n-1: a lower one is fetched for the token after it
            // (Section 3.4.2: the rule violation that is allowed "to prevent waiting")
            ++in_starts_;
            if (hot < k) ++violations_;
        }
    }
    return PIE_OK;
}

}  // namespace pie

// ------------------------------------------------------------------------------------ C ABI
using pie::Fifo;
using pie::Table;

extern "C" {

pie_table *pie_table_create(int32_t n_layers, int32_t n_logical, int64_t n_gpu_slots, int64_t n_host_slots) {
    if (n_layers <= 0 || n_logical <= 0 || n_gpu_slots < 0 || n_host_slots < 0) return nullptr;
    return reinterpret_cast<pie_table *>(new (std::nothrow) Table(n_layers, n_logical, n_gpu_slots, n_host_slots));
}
void pie_table_destroy(pie_table *t) { delete reinterpret_cast<Table *>(t); }
int pie_table_alloc(pie_table *t, int32_t block, int32_t on_host) {
    return t ? reinterpret_cast<Table *>(t)->alloc(block, on_host != 0) : PIE_ERR_INVALID;
}
int pie_table_free(pie_table *t, int32_t block) {
    return t ? reinterpret_cast<Table *>(t)->free_block(block) : PIE_ERR_INVALID;
}
int pie_table_swap(pie_table *t, int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket,
                   int32_t *moved_ids, int32_t *src_slots, int32_t *dst_slots, int64_t *n_moved, int64_t *waits) {
    if (!t || !ticket || !moved_ids || !src_slots || !dst_slots || !n_moved || !waits) return PIE_ERR_INVALID;
    return reinterpret_cast<Table *>(t)->swap(queue, layer, ids, n, ticket, moved_ids, src_slots, dst_slots, n_moved,
                                              waits);
}
int pie_table_swap_ex(pie_table *t, int32_t queue, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket,
                      int32_t *moved_ids, int32_t *src_slots, int32_t *dst_slots, uint8_t *elided, int64_t *n_moved,
                      int64_t *waits) {
    if (!t || !ticket || !moved_ids || !src_slots || !dst_slots || !elided || !n_moved || !waits) return PIE_ERR_INVALID;
    return reinterpret_cast<Table *>(t)->swap(queue, layer, ids, n, ticket, moved_ids, src_slots, dst_slots, n_moved,
                                              waits, elided);
}
int pie_table_set_retention(pie_table *t, int32_t on) {
    if (!t) return PIE_ERR_INVALID;
    reinterpret_cast<Table *>(t)->set_retain(on != 0);
    return PIE_OK;
}
int64_t pie_table_kept_copies(const pie_table *t) { return t ? reinterpret_cast<const Table *>(t)->kept_copies() : 0; }
int pie_table_drop_host_copy(pie_table *t, int32_t layer, int32_t block) {
    return t ? reinterpret_cast<Table *>(t)->drop_host_copy(layer, block) : PIE_ERR_INVALID;
}
int pie_table_mark_dirty(pie_table *t, int32_t layer, const int32_t *ids, int64_t n) {
    return t ? reinterpret_cast<Table *>(t)->mark_dirty(layer, ids, n) : PIE_ERR_INVALID;
}
int pie_table_attention(pie_table *t, int32_t layer, const int32_t *ids, int64_t n, int64_t *ticket, int64_t *waits) {
    if (!t || !ticket || !waits) return PIE_ERR_INVALID;
    return reinterpret_cast<Table *>(t)->attention(layer, ids, n, ticket, waits);
}
int pie_table_confirm(pie_table *t, int32_t queue, int64_t ticket) {
    return t ? reinterpret_cast<Table *>(t)->confirm(queue, ticket) : PIE_ERR_INVALID;
}
int pie_table_state(pie_table *t, int32_t layer, int32_t block, int32_t *state, int32_t *gpu_slot,
                    int32_t *host_slot) {
    return t ? reinterpret_cast<Table *>(t)->state(layer, block, state, gpu_slot, host_slot) : PIE_ERR_INVALID;
}
int pie_table_init_capacity(pie_table *t, int32_t size) {
    return t ? reinterpret_cast<Table *>(t)->init_capacity(size) : PIE_ERR_INVALID;
}
int pie_table_resize_begin(pie_table *t, int32_t new_size) {
    return t ? reinterpret_cast<Table *>(t)->resize_begin(new_size) : PIE_ERR_INVALID;
}
int pie_table_layer_pass(pie_table *t, int32_t layer) {
    if (!t) return PIE_ERR_INVALID;
    Table *tb = reinterpret_cast<Table *>(t);
    if (layer < 0 || layer >= tb->L) return PIE_ERR_RANGE;
    return tb->layer_pass(layer) ? 1 : 0;
}
int pie_table_capacity(pie_table *t, int32_t *visible, int32_t *alloc_limit, int32_t *target, int32_t *layers_moved) {
    if (!t) return PIE_ERR_INVALID;
    Table *tb = reinterpret_cast<Table *>(t);
    if (visible) *visible = tb->capacity();
    if (alloc_limit) *alloc_limit = tb->alloc_limit();
    if (target) *target = tb->resize_target();
    if (layers_moved) *layers_moved = tb->layers_moved();
    return PIE_OK;
}

pie_fifo *pie_fifo_create(int32_t n_layers, int32_t gpu_regions, int32_t cpu_regions, const uint8_t *on_cpu) {
    if (n_layers <= 0 || gpu_regions <= 0 || cpu_regions < 0) return nullptr;
    return reinterpret_cast<pie_fifo *>(new (std::nothrow) Fifo(n_layers, gpu_regions, cpu_regions, on_cpu));
}
void pie_fifo_destroy(pie_fifo *f) { delete reinterpret_cast<Fifo *>(f); }
int pie_fifo_complete(pie_fifo *f, int32_t dir) { return f ? reinterpret_cast<Fifo *>(f)->complete(dir) : PIE_ERR_INVALID; }
int pie_fifo_layer_start(pie_fifo *f, int32_t k, int32_t *start_out, int32_t *start_in) {
    return f ? reinterpret_cast<Fifo *>(f)->layer_start(k, start_out, start_in) : PIE_ERR_INVALID;
}
int pie_fifo_location(pie_fifo *f, int32_t layer) {
    return f ? reinterpret_cast<Fifo *>(f)->location(layer) : PIE_ERR_INVALID;
}
int pie_fifo_counters(const pie_fifo *f, int64_t *in_starts, int64_t *violations) {
    if (!f) return PIE_ERR_INVALID;
    if (in_starts) *in_starts = reinterpret_cast<const Fifo *>(f)->in_starts();
    if (violations) *violations = reinterpret_cast<const Fifo *>(f)->violations();
    return PIE_OK;
}

// state: [0] 1 + the lowest number of CPU layers known to make the computation wait (0: none), [1] windows left before
// it may be tried again, [2] the length of the next such pause (0: the first, 4; doubles up to 96).
int32_t pie_layer_controller_decide(double *state, int32_t m, int32_t m_max, double stall, double compute, int64_t in_starts,
                                    int64_t violations, double v_trigger, double eps) {
    if (v_trigger <= 0) v_trigger = 0.3;
    if (eps <= 0) eps = 0.02;
    if (state[2] <= 0) state[2] = 4;
    if (stall > eps * compute) {
        state[0] = state[0] > 0 ? std::min(state[0], 1.0 + m) : 1.0 + m;
        state[1] = state[2];
        state[2] = std::min(2.0 * state[2], 96.0);
        return std::max(0, m - 1);
    }
    const bool too_small = in_starts == 0 || (double)violations >= v_trigger * (double)in_starts;
    if (too_small && m < m_max) {
        if (state[0] > 0 && m + 1 >= (int32_t)state[0] - 1 && state[1] > 0) {
            state[1] -= 1;
            return m;
        }
        return m + 1;
    }
    return m;
}

// state[0..3]: stalled flags of the last steps (newest last), state[4]: how many are valid,
// state[5]: eps override, state[6]: u_hi override (0 = default), state[7]: steps left before the next increase.
// Constants (the paper gives none): eps = 0.02, back off on 2 stalls within 4 steps, grow while the
// link is busy for less than 0.9 of the compute time, and after an increase wait 3 steps before the next one
// (measurements arrive a few steps late: a change must be seen at work before it is built upon).
// Performance record (Section 3.4.2): the lowest ratio known to make the computation wait is remembered; a probe
// back up to it waits 3 steps after the back-off the first time and twice as long after every failed probe (at most
// 96); four unstalled steps at or above that ratio clear the record.
// state: [0..3] stall flags of the window, [4] their count, [5] eps, [6] u_hi, [7] steps left before the next increase,
// [8] 1 + the bad ratio (0: none), [9] hold, [10] steps since the last back-off, [11] unstalled steps at or above it.
double pie_controller_decide(double *state, double ratio, double step, double stall, double compute,
                             double swap_busy) {
    const double eps = state[5] > 0 ? state[5] : 0.02, u_hi = state[6] > 0 ? state[6] : 0.9;
    const int window = 4, k_dec = 2, cooldown = 3, hold_max = 96;
    int n = (int)state[4];
    bool stalled = stall > eps * compute;
    if (n == window) {
        for (int i = 1; i < window; ++i) state[i - 1] = state[i];
        n = window - 1;
    }
    state[n++] = stalled ? 1.0 : 0.0;
    state[4] = n;
    bool has_bad = state[8] > 0;
    double r_bad = state[8] - 1.0;
    if (state[9] <= 0) state[9] = cooldown;
    state[10] += 1;
    if (has_bad) {
        state[11] = (!stalled && ratio >= r_bad - 1e-12) ? state[11] + 1 : 0;
        if (state[11] >= window) {
            state[8] = 0;
            state[9] = cooldown;
            state[11] = 0;
            has_bad = false;
        }
    }
    if (stalled) {
        int count = 0;
        for (int i = 0; i < n; ++i) count += state[i] != 0.0;
        if (count >= k_dec) {
            const bool again = has_bad && ratio <= r_bad + 1e-12;
            state[9] = again ? std::min(2.0 * state[9], (double)hold_max) : (double)cooldown;
            state[8] = 1.0 + ratio;
            state[10] = 0;
            state[11] = 0;
            ratio = std::max(0.0, ratio - step);
            state[4] = 0;  // start a fresh window after a change
        }
    } else if (state[7] > 0) {
        state[7] -= 1;
    } else if (swap_busy < u_hi * compute && ratio < 1.0) {
        const double target = std::min(1.0, ratio + step);
        if (!(has_bad && target >= r_bad - 1e-12 && state[10] < state[9])) {
            ratio = target;
            state[7] = cooldown;
        }
    }
    return ratio;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Performance records against throughput (Section 3.4.2, last paragraph): a cap on the ratio from the
// throughput the serving system reports per window.  NORMAL: no cap, until a report shows no gain over the
// record one step below (the workload has stopped scaling): stop increasing and test one step lower.
// TEST_DOWN: not worse than the reference -> keep it and try lower still; worse -> one step back up, HOLD.
// HOLD: every `period` reports probe one step up.  PROBE_UP: better by more than tol -> NORMAL again, else back
// down and HOLD.  Reports at a ratio other than the cap only update the records; `patience` of them in a row
// end a test at the ratio reported.
// ---------------------------------------------------------------------------------------------
namespace {
struct Governor {
    enum { NORMAL = 0, TEST_DOWN = 1, HOLD = 2, PROBE_UP = 3 };
    static constexpr int K_MAX = 1 << 30;
    double step, tol;
    int period, patience;
    int state = NORMAL, cap = K_MAX, since = 0, off = 0;
    double ref = 0.0;
    std::map<int, double> rec;
    double cap_ratio() const { return cap >= K_MAX ? 1.0 : cap * step; }
    double report(double ratio, double throughput) {
        const int k = (int)std::llround(ratio / step);
        rec[k] = throughput;
        switch (state) {
        case NORMAL: {
            auto below = rec.find(k - 1);
            if (k > 0 && below != rec.end() && throughput <= below->second * (1 + tol)) {
                state = TEST_DOWN;
                cap = k - 1;
                ref = throughput;
                off = 0;
            }
            break;
        }
        case TEST_DOWN:
            if (k != cap) {
                if (++off >= patience) { state = HOLD; cap = k; since = 0; off = 0; }
            } else if (throughput >= ref * (1 - tol)) {
                ref = std::max(ref, throughput);
                off = 0;
                if (cap > 0) --cap;
                else { state = HOLD; since = 0; }
            } else {
                state = HOLD;
                cap = cap + 1;
                since = 0;
                off = 0;
            }
            break;
        case HOLD:
            if (++since >= period) { state = PROBE_UP; ref = throughput; cap = cap + 1; off = 0; }
            break;
        default:  // PROBE_UP
            if (k != cap) {
                if (++off >= patience) { state = HOLD; cap = k; since = 0; off = 0; }
            } else if (throughput > ref * (1 + tol)) {
                state = NORMAL;
                cap = K_MAX;
                rec.clear();
                rec[k] = throughput;
            } else {
                state = HOLD;
                cap = cap - 1;
                since = 0;
                off = 0;
            }
        }
        return cap_ratio();
    }
};
}  // namespace

extern "C" {
pie_governor *pie_governor_create(double step, double tol, int32_t period, int32_t patience) {
    if (!(step > 0)) return nullptr;
    Governor *g = new (std::nothrow) Governor();
    if (!g) return nullptr;
    g->step = step;
    g->tol = tol > 0 ? tol : 0.02;
    g->period = period > 0 ? period : 8;
    g->patience = patience > 0 ? patience : 6;
    return reinterpret_cast<pie_governor *>(g);
}
void pie_governor_destroy(pie_governor *g) { delete reinterpret_cast<Governor *>(g); }
double pie_governor_report(pie_governor *g, double ratio, double throughput) {
    return g ? reinterpret_cast<Governor *>(g)->report(ratio, throughput) : 1.0;
}
int pie_governor_state(const pie_governor *g, int32_t *state, int32_t *cap_steps) {
    if (!g) return PIE_ERR_INVALID;
    const Governor *gg = reinterpret_cast<const Governor *>(g);
    if (state) *state = gg->state;
    if (cap_steps) *cap_steps = gg->cap >= Governor::K_MAX ? -1 : gg->cap;
    return PIE_OK;
}
}
