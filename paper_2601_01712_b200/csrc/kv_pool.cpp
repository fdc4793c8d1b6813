// Paged prefix-KV pool: host metadata and tier transfers (paper Sections 3.3, 3.4).
#include "kv_pool.hpp"

#include <algorithm>

namespace relaygr {

namespace {
// Host-only backend: tiers are plain host memory and copies are synchronous.  Events complete at once, unless a test
// has switched to manual mode: then a recorded event stays pending until the test completes it, so that the states
// that need time on a GPU (LOADING, pages waiting for a spill) can be held and looked at.  Copies can be told to fail.
struct HostBackend : Backend {
    struct Ev { bool pending = false; };
    bool is_cuda() const override { return false; }
    int copy(void *dst, const void *src, size_t bytes)
    {
        if (fail_copies_ > 0) { --fail_copies_; return -1; }
        std::memcpy(dst, src, bytes);
        return 0;
    }
    int copy_h2d(void *dst, const void *src, size_t bytes, void *) override { return copy(dst, src, bytes); }
    int copy_d2h(void *dst, const void *src, size_t bytes, void *) override { return copy(dst, src, bytes); }
    void *event_create() override { return new Ev(); }
    void event_destroy(void *ev) override
    {
        pending_.erase(std::remove(pending_.begin(), pending_.end(), (Ev *)ev), pending_.end());
        delete (Ev *)ev;
    }
    int event_record(void *ev, void *) override
    {
        Ev *e = (Ev *)ev;
        pending_.erase(std::remove(pending_.begin(), pending_.end(), e), pending_.end());
        e->pending = manual_;
        if (manual_) pending_.push_back(e);
        return 0;
    }
    bool event_done(void *ev) override { return !((Ev *)ev)->pending; }
    int stream_wait(void *, void *) override { ++stream_waits_; return 0; }
    int64_t control(int32_t what, int64_t arg) override
    {
        switch (what) {
            case RELAYGR_HOSTCTL_MANUAL_EVENTS: manual_ = arg != 0; return 0;
            case RELAYGR_HOSTCTL_COMPLETE_EVENTS: {
                int64_t n = 0;
                while (!pending_.empty() && (arg < 0 || n < arg)) { pending_.front()->pending = false; pending_.erase(pending_.begin()); ++n; }
                return n;
            }
            case RELAYGR_HOSTCTL_FAIL_COPIES: fail_copies_ = arg < 0 ? 0 : arg; return 0;
            case RELAYGR_HOSTCTL_STREAM_WAITS: return stream_waits_;
            case RELAYGR_HOSTCTL_PENDING_EVENTS: return (int64_t)pending_.size();
        }
        return RELAYGR_E_INVALID;
    }
    bool manual_ = false;
    int64_t fail_copies_ = 0, stream_waits_ = 0;
    std::vector<Ev *> pending_;      // in record order
};
}  // namespace

Backend *make_host_backend() { return new HostBackend(); }

KvPool::KvPool(Backend *be, const relaygr_model_cfg &cfg, void *hbm, size_t hbm_bytes, void *host, size_t host_bytes)
    : be_(be), hbm_((char *)hbm), host_((char *)host)
{
    const size_t esize = cfg.dtype == RELAYGR_DTYPE_F32 ? 4 : 2;
    page_bytes_ = (size_t)cfg.n_layers * 2 * (size_t)cfg.page_tokens * (size_t)cfg.d_model * esize;
    n_pages_ = (int64_t)(hbm_bytes / page_bytes_);
    n_host_pages_ = host ? (int64_t)(host_bytes / page_bytes_) : 0;
    page_used_.assign((size_t)n_pages_, 0);
    page_release_.assign((size_t)n_pages_, std::vector<int64_t>());
    host_release_.assign((size_t)n_host_pages_, -1);
    free_pages_.reserve((size_t)n_pages_);
    for (int64_t p = n_pages_ - 1; p >= 0; --p) free_pages_.push_back((int32_t)p);   // pop_back hands out 0, 1, 2, ...
    free_host_.reserve((size_t)n_host_pages_);
    for (int64_t p = n_host_pages_ - 1; p >= 0; --p) free_host_.push_back((int32_t)p);
    std::memset(&st_, 0, sizeof(st_));
}

KvPool::~KvPool()
{
    for (auto &t : tickets_) if (t.ev) be_->event_destroy(t.ev);
    for (void *ev : spare_events_) be_->event_destroy(ev);
}

UserEntry *KvPool::find(uint64_t user)
{
    auto it = users_.find(user);
    return it == users_.end() ? nullptr : &it->second;
}

// ---- tickets ---------------------------------------------------------------------------------

int64_t KvPool::new_ticket(void *stream)
{
    trim_tickets();
    void *ev = nullptr;
    if (!spare_events_.empty()) { ev = spare_events_.back(); spare_events_.pop_back(); }
    else ev = be_->event_create();
    if (!ev) return -2;
    if (be_->event_record(ev, stream) != 0) { spare_events_.push_back(ev); return -2; }
    Ticket t; t.ev = ev; t.done = false;
    tickets_.push_back(t);
    return ticket_base_ + (int64_t)tickets_.size() - 1;
}

bool KvPool::ticket_done(int64_t t)
{
    if (t < ticket_base_) return true;     // includes "no ticket" (-1)
    Ticket &k = tickets_[(size_t)(t - ticket_base_)];
    if (k.done) return true;
    if (be_->event_done(k.ev)) {
        k.done = true;
        spare_events_.push_back(k.ev);
        k.ev = nullptr;
        return true;
    }
    return false;
}

void *KvPool::ticket_event(int64_t t)
{
    if (ticket_done(t)) return nullptr;
    return tickets_[(size_t)(t - ticket_base_)].ev;
}

int KvPool::wait_ticket(void *stream, int64_t t)
{
    void *ev = ticket_event(t);
    if (!ev) return 0;
    return be_->stream_wait(stream, ev);
}

void KvPool::trim_tickets()
{
    while (!tickets_.empty() && ticket_done(ticket_base_)) {
        tickets_.pop_front();
        ++ticket_base_;
    }
}

int KvPool::wait_pages_released(void *stream, const std::vector<int32_t> &pages)
{
    std::vector<int64_t> seen;
    for (int32_t p : pages) {
        std::vector<int64_t> &list = page_release_[(size_t)p];
        size_t keep = 0;
        for (int64_t t : list) {
            if (ticket_done(t)) continue;
            list[keep++] = t;
            if (std::find(seen.begin(), seen.end(), t) != seen.end()) continue;
            seen.push_back(t);
            if (wait_ticket(stream, t) != 0) return RELAYGR_E_CUDA;
        }
        list.resize(keep);
    }
    return 0;
}

int KvPool::wait_host_pages_released(void *stream, const std::vector<int32_t> &pages)
{
    std::vector<int64_t> seen;
    for (int32_t p : pages) {
        const int64_t t = host_release_[(size_t)p];
        if (t < 0) continue;
        if (ticket_done(t)) { host_release_[(size_t)p] = -1; continue; }
        if (std::find(seen.begin(), seen.end(), t) != seen.end()) continue;
        seen.push_back(t);
        if (wait_ticket(stream, t) != 0) return RELAYGR_E_CUDA;
    }
    return 0;
}

void KvPool::add_use(UserEntry &e, int64_t ticket)
{
    size_t keep = 0;
    for (int64_t t : e.use_tickets) if (!ticket_done(t)) e.use_tickets[keep++] = t;
    e.use_tickets.resize(keep);
    if (ticket >= 0) e.use_tickets.push_back(ticket);
}

std::vector<int64_t> KvPool::pending_of(UserEntry &e)
{
    std::vector<int64_t> out;
    if (e.ready_ticket >= 0 && !ticket_done(e.ready_ticket)) out.push_back(e.ready_ticket);
    for (int64_t t : e.use_tickets) if (!ticket_done(t) && std::find(out.begin(), out.end(), t) == out.end()) out.push_back(t);
    return out;
}

int KvPool::wait_pages_of(uint64_t user, void *stream, std::string &err)
{
    UserEntry *e = find(user);
    if (!e) { err = "kv_wait_pages: unknown user"; return RELAYGR_E_MISS; }
    if (wait_pages_released(stream, e->pages) != 0) { err = "kv_wait_pages: could not make the stream wait"; return RELAYGR_E_CUDA; }
    return 0;
}

// ---- pages -----------------------------------------------------------------------------------

int KvPool::take_pages(int32_t n, const int32_t *ids, std::vector<int32_t> &out, std::string &err)
{
    out.clear();
    if (ids) {
        for (int32_t i = 0; i < n; ++i) {
            const int32_t p = ids[i];
            if (p < 0 || p >= n_pages_ || page_used_[(size_t)p]) {
                for (int32_t q : out) page_used_[(size_t)q] = 0;
                out.clear();
                err = "kv_alloc: page id out of range, in use or repeated";
                return p < 0 || p >= n_pages_ ? RELAYGR_E_INVALID : RELAYGR_E_NOSPACE;
            }
            page_used_[(size_t)p] = 1;
            out.push_back(p);
        }
        // the free list is rebuilt lazily: used pages are skipped when popped
        return 0;
    }
    // count what is really free (entries of the list may have been taken by id)
    std::vector<int32_t> got;
    while ((int32_t)got.size() < n && !free_pages_.empty()) {
        const int32_t p = free_pages_.back();
        free_pages_.pop_back();
        if (page_used_[(size_t)p]) continue;     // stale: taken by explicit id meanwhile
        page_used_[(size_t)p] = 1;
        got.push_back(p);
    }
    if ((int32_t)got.size() < n) {
        for (auto it = got.rbegin(); it != got.rend(); ++it) { page_used_[(size_t)*it] = 0; free_pages_.push_back(*it); }
        err = "not enough free pages in the HBM pool";
        return RELAYGR_E_NOSPACE;
    }
    out.swap(got);
    return 0;
}

void KvPool::release_pages(std::vector<int32_t> &pages, const std::vector<int64_t> &behind)
{
    for (auto it = pages.rbegin(); it != pages.rend(); ++it) {
        page_used_[(size_t)*it] = 0;
        // what an earlier owner left pending stays: the entry that releases now may never have run anything on the page
        std::vector<int64_t> &list = page_release_[(size_t)*it];
        size_t keep = 0;
        for (int64_t t : list) if (!ticket_done(t)) list[keep++] = t;
        list.resize(keep);
        for (int64_t t : behind)
            if (t >= 0 && !ticket_done(t) && std::find(list.begin(), list.end(), t) == list.end()) list.push_back(t);
        free_pages_.push_back(*it);
    }
    pages.clear();
    // a page taken by id and released again may now sit twice in the list; the copy that is popped
    // second sees page_used_ == 1 or is skipped as a duplicate free, so compact when the list grows
    if ((int64_t)free_pages_.size() > 2 * n_pages_) {
        std::vector<uint8_t> seen((size_t)n_pages_, 0);
        std::vector<int32_t> keep;
        for (int32_t p : free_pages_) if (!page_used_[(size_t)p] && !seen[(size_t)p]) { seen[(size_t)p] = 1; keep.push_back(p); }
        free_pages_.swap(keep);
    }
}

void KvPool::release_host_pages(std::vector<int32_t> &pages, int64_t behind)
{
    for (int32_t p : pages) {
        host_release_[(size_t)p] = (behind >= 0 && !ticket_done(behind)) ? behind : -1;
        free_host_.push_back(p);
    }
    pages.clear();
}

int KvPool::copy_pages(bool to_host, const std::vector<int32_t> &dev, const std::vector<int32_t> &host, void *stream)
{
    // consecutive pages on both sides are merged into one copy
    size_t i = 0;
    const size_t n = dev.size();
    while (i < n) {
        size_t j = i + 1;
        while (j < n && dev[j] == dev[j - 1] + 1 && host[j] == host[j - 1] + 1) ++j;
        char *d = hbm_ + (size_t)dev[i] * page_bytes_;
        char *h = host_ + (size_t)host[i] * page_bytes_;
        const size_t bytes = (j - i) * page_bytes_;
        const int rc = to_host ? be_->copy_d2h(h, d, bytes, stream) : be_->copy_h2d(d, h, bytes, stream);
        if (rc != 0) return RELAYGR_E_CUDA;
        i = j;
    }
    return 0;
}

// ---- user operations ---------------------------------------------------------------------------

int KvPool::alloc(uint64_t user, int32_t prefix_len, const int32_t *page_ids, std::string &err)
{
    if (prefix_len < 1) { err = "kv_alloc: prefix_len must be >= 1"; return RELAYGR_E_INVALID; }
    if (users_.count(user)) { err = "kv_alloc: user already has an entry"; return RELAYGR_E_EXISTS; }
    const int32_t n = (prefix_len + 63) / 64;
    UserEntry e;
    e.state = UserState::Allocated;
    e.prefix_len = prefix_len;
    const int rc = take_pages(n, page_ids, e.pages, err);
    if (rc != 0) return rc;
    users_.emplace(user, std::move(e));
    return 0;
}

int32_t KvPool::tier_of(UserEntry &e)
{
    if (e.state == UserState::Loading && ticket_done(e.ready_ticket)) e.state = UserState::Resident;
    switch (e.state) {
        case UserState::Allocated: return RELAYGR_TIER_ALLOCATED;
        case UserState::Resident: return RELAYGR_TIER_HBM;
        case UserState::Loading: return RELAYGR_TIER_LOADING;
        case UserState::Host: return RELAYGR_TIER_HOST;
    }
    return RELAYGR_TIER_MISS;
}

int KvPool::free_user(uint64_t user, std::string &err)
{
    UserEntry *e = find(user);
    if (!e) { err = "kv_free: unknown user"; return RELAYGR_E_MISS; }
    if (tier_of(*e) == RELAYGR_TIER_LOADING) { err = "kv_free: reload in flight"; return RELAYGR_E_BUSY; }
    release_pages(e->pages, pending_of(*e));
    release_host_pages(e->host_pages, e->host_ticket);      // a spill copy may still be writing them
    users_.erase(user);
    return 0;
}

int KvPool::evict(uint64_t user, bool spill, void *side, std::string &err)
{
    UserEntry *e = find(user);
    if (!e) { err = "kv_evict: unknown user"; return RELAYGR_E_MISS; }
    const int32_t tier = tier_of(*e);
    if (tier == RELAYGR_TIER_LOADING) { err = "kv_evict: reload in flight"; return RELAYGR_E_BUSY; }
    if (tier == RELAYGR_TIER_HOST) { err = "kv_evict: user holds no HBM pages"; return RELAYGR_E_MISS; }
    if (tier == RELAYGR_TIER_ALLOCATED) {            // nothing was computed yet: just give the pages back
        release_pages(e->pages, pending_of(*e));
        users_.erase(user);
        return 0;
    }
    std::vector<int64_t> release_after = pending_of(*e);
    if (spill && e->host_pages.empty()) {
        if (!host_ || (int64_t)free_host_.size() < (int64_t)e->pages.size()) {
            err = "kv_evict: host tier is full or absent";
            return RELAYGR_E_NOSPACE;
        }
        std::vector<int32_t> hp;
        for (size_t i = 0; i < e->pages.size(); ++i) { hp.push_back(free_host_.back()); free_host_.pop_back(); }
        // the copy runs after the producer and every enqueued reader of these pages, and after whatever may still be
        // writing the host pages it lands in
        int rc = 0;
        for (int64_t t : release_after) if (rc == 0) rc = wait_ticket(side, t);
        if (rc == 0) rc = wait_host_pages_released(side, hp);
        if (rc == 0) rc = copy_pages(true, e->pages, hp, side);
        const int64_t t = rc == 0 ? new_ticket(side) : -2;
        if (rc != 0 || t == -2) {
            for (auto it = hp.rbegin(); it != hp.rend(); ++it) free_host_.push_back(*it);
            err = "kv_evict: spill copy could not be enqueued";
            return RELAYGR_E_CUDA;
        }
        e->host_pages.swap(hp);
        e->host_ticket = t;
        release_after.assign(1, t);                   // recorded behind everything the copy waited for
        st_.spills += 1;
        st_.spill_bytes += (int64_t)(e->host_pages.size() * page_bytes_);
    }
    release_pages(e->pages, release_after);
    if (e->host_pages.empty()) {
        users_.erase(user);
    } else {
        e->state = UserState::Host;
        e->ready_ticket = -1;
        e->use_tickets.clear();
    }
    return 0;
}

int KvPool::reload(uint64_t user, void *side, void **ready_out, std::string &err)
{
    if (ready_out) *ready_out = nullptr;
    UserEntry *e = find(user);
    if (!e) { st_.misses += 1; err = "kv_reload: unknown user"; return RELAYGR_E_MISS; }
    const int32_t tier = tier_of(*e);
    if (tier == RELAYGR_TIER_ALLOCATED) { err = "kv_reload: user was never pre-inferred"; return RELAYGR_E_MISS; }
    if (tier == RELAYGR_TIER_HBM || tier == RELAYGR_TIER_LOADING) {     // idempotent / single-flight
        if (ready_out) *ready_out = ticket_event(e->ready_ticket);
        return 0;
    }
    // HOST: bounded number of reloads in flight
    int32_t inflight = 0;
    for (auto &kv : users_) if (kv.second.state == UserState::Loading && tier_of(kv.second) == RELAYGR_TIER_LOADING) ++inflight;
    if (inflight >= max_inflight_) { err = "kv_reload: too many reloads in flight"; return RELAYGR_E_BUSY; }
    std::vector<int32_t> pages;
    int rc = take_pages((int32_t)e->host_pages.size(), nullptr, pages, err);
    if (rc != 0) return rc;
    rc = wait_pages_released(side, pages);
    if (rc == 0) rc = wait_ticket(side, e->host_ticket);
    if (rc == 0) rc = copy_pages(false, pages, e->host_pages, side);
    const int64_t t = rc == 0 ? new_ticket(side) : -2;
    if (rc != 0 || t == -2) {
        // the user stays in HOST; the pages go back, still behind whatever their earlier owners left pending, and behind
        // the part of this reload that may have been enqueued
        std::vector<int64_t> behind;
        const int64_t tf = new_ticket(side);
        if (tf >= 0) behind.push_back(tf);
        release_pages(pages, behind);
        err = "kv_reload: copy could not be enqueued";
        return RELAYGR_E_CUDA;
    }
    e->pages.swap(pages);
    e->ready_ticket = t;
    e->use_tickets.clear();
    e->state = UserState::Loading;
    st_.reloads += 1;
    st_.reload_bytes += (int64_t)(e->pages.size() * page_bytes_);
    if (ready_out) *ready_out = ticket_event(t);
    return 0;
}

void KvPool::count_hit(int32_t tier)
{
    switch (tier) {
        case RELAYGR_TIER_HBM: st_.hits_hbm += 1; break;
        case RELAYGR_TIER_LOADING: st_.hits_loading += 1; break;
        case RELAYGR_TIER_HOST: st_.hits_host += 1; break;
        default: st_.misses += 1; break;
    }
}

int KvPool::lookup(uint64_t user, int32_t *tier, int32_t *prefix_len, bool count)
{
    UserEntry *e = find(user);
    const int32_t t = e ? tier_of(*e) : RELAYGR_TIER_MISS;
    if (tier) *tier = t;
    if (prefix_len) *prefix_len = e ? e->prefix_len : 0;
    if (count) count_hit(t);
    return 0;
}

int KvPool::pages_of(uint64_t user, int32_t *out, int32_t cap, int32_t *n_out, std::string &err)
{
    UserEntry *e = find(user);
    if (!e) { err = "kv_pages: unknown user"; return RELAYGR_E_MISS; }
    if (n_out) *n_out = (int32_t)e->pages.size();
    if (out) {
        if (cap < (int32_t)e->pages.size()) { err = "kv_pages: output too small"; return RELAYGR_E_INVALID; }
        std::copy(e->pages.begin(), e->pages.end(), out);
    }
    return 0;
}

void KvPool::stats(relaygr_pool_stats *out)
{
    relaygr_pool_stats s = st_;
    s.pages_total = n_pages_;
    int64_t used = 0;
    for (uint8_t u : page_used_) used += u;
    s.pages_free = n_pages_ - used;
    s.host_pages_total = n_host_pages_;
    s.host_pages_free = (int64_t)free_host_.size();
    s.users_hbm = s.users_loading = s.users_host = s.users_allocated = 0;
    for (auto &kv : users_) {
        switch (tier_of(kv.second)) {
            case RELAYGR_TIER_HBM: s.users_hbm += 1; break;
            case RELAYGR_TIER_LOADING: s.users_loading += 1; break;
            case RELAYGR_TIER_HOST: s.users_host += 1; break;
            case RELAYGR_TIER_ALLOCATED: s.users_allocated += 1; break;
        }
    }
    *out = s;
}

}  // namespace relaygr
