// Host-side metadata of the paged prefix-KV pool: page allocator, user map, the
// per-user state machine and the ordering tickets that make page reuse safe.
// Device work (copies, events) goes through a small backend interface so that the
// same logic runs against CUDA or, for host-only contexts, against plain memcpy.
#pragma once

#include <cstdint>
#include <cstring>
#include <deque>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/relaygr.h"

namespace relaygr {

// Backend: how bytes move between the tiers and how completion is tracked.
struct Backend {
    virtual ~Backend() {}
    virtual bool is_cuda() const = 0;
    virtual int copy_h2d(void *dst, const void *src, size_t bytes, void *stream) = 0;
    virtual int copy_d2h(void *dst, const void *src, size_t bytes, void *stream) = 0;
    virtual void *event_create() = 0;                 // nullptr on failure
    virtual void event_destroy(void *ev) = 0;
    virtual int event_record(void *ev, void *stream) = 0;
    virtual bool event_done(void *ev) = 0;
    virtual int stream_wait(void *stream, void *ev) = 0;
    // Test control (host backend only; see relaygr_kv_host_backend_control).  Returns a negative status when unsupported.
    virtual int64_t control(int32_t what, int64_t arg) { (void)what; (void)arg; return RELAYGR_E_UNSUPPORTED; }
};

Backend *make_cuda_backend();
Backend *make_host_backend();

enum class UserState : int32_t { Allocated = 1, Resident = 2, Loading = 3, Host = 4 };

struct UserEntry {
    UserState state;
    int32_t prefix_len;
    std::vector<int32_t> pages;       // HBM page ids, logical order (empty when Host)
    std::vector<int32_t> host_pages;  // host-tier page ids (empty when no host copy)
    int64_t ready_ticket = -1;        // producer of the HBM copy (pre-infer, commit or reload)
    std::vector<int64_t> use_tickets; // enqueued readers of the HBM pages that may still be running (any stream)
    int64_t host_ticket = -1;         // spill copy that fills the host pages
};

// A ticket stands for "everything enqueued up to this point on some stream".
struct Ticket {
    void *ev = nullptr;
    bool done = false;
};

class KvPool {
public:
    KvPool(Backend *be, const relaygr_model_cfg &cfg, void *hbm, size_t hbm_bytes, void *host, size_t host_bytes);
    ~KvPool();

    size_t page_bytes() const { return page_bytes_; }
    int64_t n_pages() const { return n_pages_; }
    void *slab() const { return hbm_; }
    Backend *backend() const { return be_; }

    int alloc(uint64_t user, int32_t prefix_len, const int32_t *page_ids, std::string &err);
    int free_user(uint64_t user, std::string &err);
    int evict(uint64_t user, bool spill, void *side, std::string &err);
    int reload(uint64_t user, void *side, void **ready_out, std::string &err);
    int lookup(uint64_t user, int32_t *tier, int32_t *prefix_len, bool count);
    int pages_of(uint64_t user, int32_t *out, int32_t cap, int32_t *n_out, std::string &err);
    void stats(relaygr_pool_stats *out);
    void set_max_inflight(int32_t n) { max_inflight_ = n < 1 ? 1 : n; }

    UserEntry *find(uint64_t user);
    // Current tier of an entry, promoting Loading -> Resident when its reload has completed.
    int32_t tier_of(UserEntry &e);

    // Ordering helpers used by the compute calls.
    int64_t new_ticket(void *stream);                  // records an event on stream; -2 on failure
    bool ticket_done(int64_t t);
    void *ticket_event(int64_t t);                     // nullptr when done / unknown
    int wait_ticket(void *stream, int64_t t);          // make stream wait for t (no-op if done)
    int wait_pages_released(void *stream, const std::vector<int32_t> &pages);
    void add_use(UserEntry &e, int64_t ticket);        // remember a reader of the user's HBM pages
    int wait_pages_of(uint64_t user, void *stream, std::string &err);
    void count_hit(int32_t tier);

private:
    int take_pages(int32_t n, const int32_t *ids, std::vector<int32_t> &out, std::string &err);
    // Every ticket that must complete before the user's HBM pages may be overwritten: producer, readers, spill copy.
    std::vector<int64_t> pending_of(UserEntry &e);
    void release_pages(std::vector<int32_t> &pages, const std::vector<int64_t> &behind);
    void release_host_pages(std::vector<int32_t> &pages, int64_t behind);
    int wait_host_pages_released(void *stream, const std::vector<int32_t> &pages);
    void trim_tickets();
    int copy_pages(bool to_host, const std::vector<int32_t> &dev, const std::vector<int32_t> &host, void *stream);

    Backend *be_;
    size_t page_bytes_;
    char *hbm_;
    char *host_;
    int64_t n_pages_, n_host_pages_;
    std::vector<int32_t> free_pages_, free_host_;
    std::vector<uint8_t> page_used_;
    // per HBM page: reuse only behind ALL of these tickets (a page may change hands while the copy or the kernels of an
    // earlier owner are still running, so one ticket per page is not enough)
    std::vector<std::vector<int64_t>> page_release_;
    std::vector<int64_t> host_release_;               // per host page: the spill copy that may still be writing it
    std::unordered_map<uint64_t, UserEntry> users_;
    std::deque<Ticket> tickets_;
    int64_t ticket_base_ = 0;
    std::vector<void *> spare_events_;
    int32_t max_inflight_ = 8;
    relaygr_pool_stats st_;
};

}  // namespace relaygr
