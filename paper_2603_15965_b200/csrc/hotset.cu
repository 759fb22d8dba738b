// Hot-set slot table (Definition 5.1, Eq. 10-11): S adapter slots of fixed-address stacks A_hot[S, M, d, r] and
// B_hot[S, M, r, d], a slot table sigma : [S] -> adapters maintained off the critical path, and its inverse on the
// device (adapter id -> slot, -1 = not resident) that the compositional router reads.
//
// This file is host bookkeeping plus asynchronous copies on a maintenance stream; the compute path never waits for it:
//   - routing reads the device table; an adapter becomes routable only when the table entry is written, which the
//     maintenance stream does AFTER the slot's weights (stream order);
//   - a slot is never refilled while it is pinned (a step that routed tokens to it is still in flight) -- the caller
//     pins the adapters of a step before it enqueues the step and unpins them when the step's event has completed;
//   - eviction picks the least recently pinned unpinned slot; the table entry of the evicted adapter is cleared on the
//     maintenance stream before the weights are overwritten.
// Copies and events go through a small backend table so that the logic can be tested on the CPU against a fake stream.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "common.cuh"

using namespace molora;

namespace {

enum SlotState : int32_t { kFree = 0, kLoading = 1, kPending = 2, kReady = 3 };   // pending: copies enqueued, event not yet done

struct Slot {
    int32_t adapter = -1;
    int32_t state = kFree;
    int32_t pins = 0;
    uint64_t last_use = 0;
    void* event = nullptr;       // backend event recorded after the slot's copies and its table update
};

molora_status_t cuda_copy_h2d(void* dst, const void* src, size_t bytes, void* stream, void*)
{
    return cuda_ok(cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, static_cast<cudaStream_t>(stream)));
}
molora_status_t cuda_event_record(void** event, void* stream, void*)
{
    if (*event == nullptr) {
        cudaEvent_t e;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return MOLORA_ERR_CUDA;
        *event = e;
    }
    return cuda_ok(cudaEventRecord(static_cast<cudaEvent_t>(*event), static_cast<cudaStream_t>(stream)));
}
int32_t cuda_event_done(void* event, void*) { return cudaEventQuery(static_cast<cudaEvent_t>(event)) == cudaSuccess ? 1 : 0; }
void cuda_event_destroy(void* event, void*)
{
    if (event != nullptr) cudaEventDestroy(static_cast<cudaEvent_t>(event));
}

}  // namespace

struct molora_hotset {
    int32_t S = 0, M = 0, n_catalog = 0;
    int32_t* table_dev = nullptr;            // device int32[n_catalog]: adapter id -> slot, -1 = not resident (caller-owned)
    std::vector<int32_t> stage;              // host words the table updates are copied from: [0] = -1, [1 + s] = s
    std::vector<Slot> slots;
    std::vector<int32_t> slot_of;            // host mirror of the table as it will be once the enqueued updates ran
    molora_hotset_backend_t be{};
    uint64_t tick = 0;
    std::mutex mu;
};

extern "C" {

molora_status_t molora_hotset_create(int32_t S, int32_t M, int32_t n_catalog, int32_t* table_dev,
                                     const molora_hotset_backend_t* backend, molora_hotset_t** out)
{
    if (out == nullptr || S < 1 || M < 1 || n_catalog < 1 || table_dev == nullptr) return MOLORA_ERR_INVALID_ARG;
    if ((int64_t)S * M > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;      // routing targets slot * M + m stay below 256
    molora_hotset* h = new (std::nothrow) molora_hotset;
    if (h == nullptr) return MOLORA_ERR_INVALID_ARG;
    h->S = S;
    h->M = M;
    h->n_catalog = n_catalog;
    h->table_dev = table_dev;
    h->slots.resize(S);
    h->slot_of.assign(n_catalog, -1);
    h->stage.resize(S + 1);
    h->stage[0] = -1;
    for (int s = 0; s < S; ++s) h->stage[1 + s] = s;
    if (backend != nullptr) h->be = *backend;
    if (h->be.copy_h2d == nullptr) h->be.copy_h2d = cuda_copy_h2d;
    if (h->be.event_record == nullptr) h->be.event_record = cuda_event_record;
    if (h->be.event_done == nullptr) h->be.event_done = cuda_event_done;
    if (h->be.event_destroy == nullptr) h->be.event_destroy = cuda_event_destroy;
    *out = h;
    return MOLORA_OK;
}

void molora_hotset_destroy(molora_hotset_t* h)
{
    if (h == nullptr) return;
    for (Slot& s : h->slots) h->be.event_destroy(s.event, h->be.user);
    delete h;
}

// Promote slots whose copies have completed (never blocks).
static void poll_locked(molora_hotset* h)
{
    for (Slot& s : h->slots)
        if (s.state == kPending && s.event != nullptr && h->be.event_done(s.event, h->be.user)) s.state = kReady;
}

int32_t molora_hotset_slot_of(molora_hotset_t* h, int32_t adapter)
{
    if (h == nullptr || adapter < 0 || adapter >= h->n_catalog) return -1;
    std::lock_guard<std::mutex> lock(h->mu);
    poll_locked(h);
    const int32_t s = h->slot_of[adapter];
    return s >= 0 && h->slots[s].state == kReady ? s : -1;
}

int32_t molora_hotset_adapter_in(molora_hotset_t* h, int32_t slot)
{
    if (h == nullptr || slot < 0 || slot >= h->S) return -1;
    std::lock_guard<std::mutex> lock(h->mu);
    return h->slots[slot].adapter;
}

molora_status_t molora_hotset_pin(molora_hotset_t* h, int32_t adapter, int32_t* slot_out)
{
    if (h == nullptr || slot_out == nullptr || adapter < 0 || adapter >= h->n_catalog) return MOLORA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(h->mu);
    poll_locked(h);
    const int32_t s = h->slot_of[adapter];
    if (s < 0 || h->slots[s].state != kReady) {
        *slot_out = -1;
        return MOLORA_ERR_NOT_RESIDENT;
    }
    ++h->slots[s].pins;
    h->slots[s].last_use = ++h->tick;
    *slot_out = s;
    return MOLORA_OK;
}

molora_status_t molora_hotset_unpin(molora_hotset_t* h, int32_t slot)
{
    if (h == nullptr || slot < 0 || slot >= h->S) return MOLORA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(h->mu);
    if (h->slots[slot].pins <= 0) return MOLORA_ERR_INVALID_ARG;
    --h->slots[slot].pins;
    return MOLORA_OK;
}

molora_status_t molora_hotset_begin_load(molora_hotset_t* h, int32_t adapter, void* maintenance_stream, int32_t* slot_out,
                                         int32_t* fresh_out, int32_t* evicted_out)
{
    if (h == nullptr || slot_out == nullptr || fresh_out == nullptr || adapter < 0 || adapter >= h->n_catalog)
        return MOLORA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(h->mu);
    poll_locked(h);
    if (evicted_out != nullptr) *evicted_out = -1;
    *fresh_out = 0;
    if (h->slot_of[adapter] >= 0) {                 // resident, or already on its way: nothing to upload
        *slot_out = h->slot_of[adapter];
        return MOLORA_OK;
    }
    int victim = -1;
    for (int s = 0; s < h->S && victim < 0; ++s)
        if (h->slots[s].state == kFree) victim = s;
    if (victim < 0) {                               // least recently pinned among the slots nothing is using
        for (int s = 0; s < h->S; ++s)
            if (h->slots[s].state == kReady && h->slots[s].pins == 0 &&
                (victim < 0 || h->slots[s].last_use < h->slots[victim].last_use))
                victim = s;
    }
    if (victim < 0) {
        *slot_out = -1;
        return MOLORA_ERR_BUSY;                     // every slot is pinned or being filled: try again later
    }
    Slot& sl = h->slots[victim];
    if (sl.adapter >= 0) {
        // the evicted adapter stops being routable before its weights are overwritten (stream order)
        const molora_status_t st = h->be.copy_h2d(h->table_dev + sl.adapter, &h->stage[0], sizeof(int32_t), maintenance_stream, h->be.user);
        if (st != MOLORA_OK) return st;
        h->slot_of[sl.adapter] = -1;
        if (evicted_out != nullptr) *evicted_out = sl.adapter;
    }
    sl.adapter = adapter;
    sl.state = kLoading;
    sl.pins = 0;
    sl.last_use = ++h->tick;                        // a fresh slot is not the next victim
    h->slot_of[adapter] = victim;
    *slot_out = victim;
    *fresh_out = 1;
    return MOLORA_OK;
}

molora_status_t molora_hotset_upload(molora_hotset_t* h, int32_t slot, void* stack_dev, const void* weights_host,
                                     size_t bytes_per_slot, void* maintenance_stream)
{
    if (h == nullptr || slot < 0 || slot >= h->S || stack_dev == nullptr || weights_host == nullptr || bytes_per_slot == 0)
        return MOLORA_ERR_INVALID_ARG;
    {
        std::lock_guard<std::mutex> lock(h->mu);
        if (h->slots[slot].state != kLoading) return MOLORA_ERR_INVALID_ARG;      // only a slot handed out by begin_load
    }
    return h->be.copy_h2d(static_cast<char*>(stack_dev) + (size_t)slot * bytes_per_slot, weights_host, bytes_per_slot,
                          maintenance_stream, h->be.user);
}

molora_status_t molora_hotset_commit(molora_hotset_t* h, int32_t slot, void* maintenance_stream)
{
    if (h == nullptr || slot < 0 || slot >= h->S) return MOLORA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(h->mu);
    Slot& sl = h->slots[slot];
    if (sl.state != kLoading) return MOLORA_ERR_INVALID_ARG;
    // after the weights (stream order): the table entry that makes the adapter routable, then the event that tells the
    // host that both have landed
    molora_status_t st = h->be.copy_h2d(h->table_dev + sl.adapter, &h->stage[1 + slot], sizeof(int32_t), maintenance_stream, h->be.user);
    if (st == MOLORA_OK) st = h->be.event_record(&sl.event, maintenance_stream, h->be.user);
    if (st != MOLORA_OK) return st;
    sl.state = kPending;
    return MOLORA_OK;
}

molora_status_t molora_route_hotset(const int32_t* ids, const int32_t* adapter_id, int64_t N, const int32_t* breaks, int32_t M,
                                    const int32_t* slot_table_dev, int32_t n_catalog, int32_t S, int32_t* r_out,
                                    uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX) return MOLORA_ERR_INVALID_ARG;
    if (M < 1 || S < 1 || n_catalog < 1) return MOLORA_ERR_INVALID_ARG;
    if ((int64_t)M * S > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (breaks == nullptr || slot_table_dev == nullptr || (N > 0 && (ids == nullptr || adapter_id == nullptr || r_out == nullptr)))
        return MOLORA_ERR_INVALID_ARG;
    return launch_route_vocab(ids, N, breaks, M, adapter_id, S, r_out, dev_status, static_cast<cudaStream_t>(stream), slot_table_dev,
                              n_catalog);
}

}  // extern "C"
