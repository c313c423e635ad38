// Scratch buffers for calls that need device memory beyond their inputs and outputs (the int8
// operand images of the INT4 pre-pass), handed out per CUDA stream.
//
// Policy, independent of CUDA so that it can be exercised on a CPU with a fake backend:
//   * a buffer last used on stream s goes to the next call on s that it is large enough for:
//     stream order keeps the two calls apart;
//   * a buffer whose last use has completed (its event reports so) may move to another stream;
//   * otherwise a new buffer is allocated, stream-ordered on s (no device-wide synchronisation);
//     a buffer of stream s that has become too small is freed the same way, after s's earlier work;
//   * while a stream is being captured into a graph nothing can be allocated and no event can
//     tell when the captured work will run, so the call takes the best buffer there is and
//     marks it "shared": it then stays with whoever holds it (as a single workspace per device
//     would), and keeping replays of that graph apart from other calls is the caller's job;
//   * two host threads never hold the same buffer at once (a buffer is leased from acquire()
//     to release(), which brackets the launches that use it).
//
// Backend concept:
//   using Stream = ...; using Event = ...;
//   int  alloc(void** p, size_t bytes, Stream s);   // stream-ordered; 0 = ok
//   int  free_after(void* p, Stream s);             // free once s has passed this point
//   int  free_now(void* p);                         // synchronous free (release_all)
//   int  event_create(Event* e); void event_destroy(Event e);
//   int  event_record(Event e, Stream s);
//   bool event_done(Event e);                       // true if never recorded
//   bool capturing(Stream s);
//   int  clear(void* p, size_t bytes, Stream s);    // stream-ordered memset to zero
#pragma once

#include <stddef.h>

#include <mutex>
#include <vector>

namespace b200gemm {

template <class Backend>
class WorkspacePool {
 public:
  using Stream = typename Backend::Stream;
  using Event = typename Backend::Event;

  struct Lease {
    void* ptr = nullptr;     // start of the buffer: `head_bytes` of zero-initialised bookkeeping
    size_t bytes = 0;        // capacity after the head
    size_t head_bytes = 0;
    int slot = -1;
  };

  explicit WorkspacePool(Backend backend = Backend()) : backend_(backend) {}

  // A buffer with at least `need` bytes behind a head of at least `head` bytes that was
  // zeroed when the buffer was allocated (and is never cleared again by the pool: whatever
  // lives there must leave it consistent).  0 = ok, else the backend's error code;
  // kNoAllocInCapture when the stream is being captured and no buffer is large enough.
  static constexpr int kNoAllocInCapture = -1000;
  int acquire(Stream s, size_t need, size_t head, Lease* out) {
    std::lock_guard<std::mutex> lock(mutex_);
    const bool cap = backend_.capturing(s);
    int pick = -1;
    // 1. this stream's own buffer
    for (size_t i = 0; i < entries_.size() && pick < 0; ++i) {
      Entry& e = entries_[i];
      if (!e.leased && e.stream == s && fits(e, need, head)) pick = static_cast<int>(i);
    }
    // 2. a buffer nobody is using any more (not asked during capture: querying an event is
    //    not allowed then, and says nothing about when the captured work will run)
    for (size_t i = 0; i < entries_.size() && pick < 0 && !cap; ++i) {
      Entry& e = entries_[i];
      if (!e.leased && !e.shared && fits(e, need, head) && backend_.event_done(e.event))
        pick = static_cast<int>(i);
    }
    if (pick < 0 && cap) {
      // 3. capture: any buffer that fits, from now on shared
      for (size_t i = 0; i < entries_.size() && pick < 0; ++i)
        if (!entries_[i].leased && fits(entries_[i], need, head)) pick = static_cast<int>(i);
      if (pick < 0) return kNoAllocInCapture;
    }
    if (pick < 0) {
      // 4. grow this stream's buffer, or add one
      int mine = -1;
      for (size_t i = 0; i < entries_.size() && mine < 0; ++i)
        if (!entries_[i].leased && !entries_[i].shared && entries_[i].ptr && entries_[i].stream == s)
          mine = static_cast<int>(i);
      for (size_t i = 0; i < entries_.size() && mine < 0; ++i)  // or an emptied slot
        if (!entries_[i].leased && !entries_[i].ptr) mine = static_cast<int>(i);
      // a replacement is never smaller than what it replaces, in either part
      if (mine >= 0 && entries_[mine].ptr) {
        if (entries_[mine].bytes > need) need = entries_[mine].bytes;
        if (entries_[mine].head_bytes > head) head = entries_[mine].head_bytes;
      }
      Entry fresh;
      int rc = backend_.alloc(&fresh.ptr, head + need, s);
      if (rc != 0) return rc;
      rc = backend_.clear(fresh.ptr, head, s);
      if (rc != 0) {
        backend_.free_after(fresh.ptr, s);
        return rc;
      }
      fresh.bytes = need;
      fresh.head_bytes = head;
      if (mine >= 0) {
        Entry& old = entries_[mine];
        // s's earlier launches may still read the old buffer
        rc = old.ptr ? backend_.free_after(old.ptr, s) : 0;
        if (rc != 0) {
          backend_.free_after(fresh.ptr, s);
          return rc;
        }
        old.ptr = fresh.ptr;
        old.bytes = fresh.bytes;
        old.head_bytes = fresh.head_bytes;
        pick = mine;
      } else {
        rc = backend_.event_create(&fresh.event);
        if (rc != 0) {
          backend_.free_after(fresh.ptr, s);
          return rc;
        }
        entries_.push_back(fresh);
        pick = static_cast<int>(entries_.size()) - 1;
      }
    }
    Entry& e = entries_[pick];
    e.leased = true;
    e.stream = s;
    if (cap) e.shared = true;
    out->ptr = e.ptr;
    out->bytes = e.bytes;
    out->head_bytes = e.head_bytes;
    out->slot = pick;
    return 0;
  }

  // The launches that use the lease have been enqueued on s.
  int release(const Lease& lease, Stream s) {
    std::lock_guard<std::mutex> lock(mutex_);
    if (lease.slot < 0 || lease.slot >= static_cast<int>(entries_.size())) return 0;
    Entry& e = entries_[lease.slot];
    e.leased = false;
    if (backend_.capturing(s)) {
      e.shared = true;
      return 0;
    }
    return backend_.event_record(e.event, s);
  }

  // Frees every buffer that is not leased right now (its slot stays, empty, for reuse, so that
  // leases handed out earlier keep their slot numbers).  The caller has synchronised the device.
  int release_all() {
    std::lock_guard<std::mutex> lock(mutex_);
    int rc = 0;
    for (Entry& e : entries_) {
      if (e.leased || !e.ptr) continue;
      const int r = backend_.free_now(e.ptr);
      if (r != 0) rc = r;
      e.ptr = nullptr;
      e.bytes = 0;
      e.head_bytes = 0;
      e.shared = false;
    }
    return rc;
  }

  size_t buffers() {
    std::lock_guard<std::mutex> lock(mutex_);
    size_t n = 0;
    for (const Entry& e : entries_) n += e.ptr ? 1 : 0;
    return n;
  }

 private:
  struct Entry {
    void* ptr = nullptr;
    size_t bytes = 0;
    size_t head_bytes = 0;
    Stream stream = Stream();
    Event event = Event();
    bool leased = false;
    bool shared = false;
  };
  static bool fits(const Entry& e, size_t need, size_t head) {
    return e.ptr && e.bytes >= need && e.head_bytes >= head;
  }

  Backend backend_;
  std::mutex mutex_;
  std::vector<Entry> entries_;
};

}  // namespace b200gemm
