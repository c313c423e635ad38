// CPU exercise of the scratch-buffer pool's policy with a fake backend (no CUDA): which
// buffer a (stream, size) request gets, when something is allocated or freed, and what stream
// capture changes.  Prints "ok" or the first failed expectation.
#include <stdio.h>
#include <stdlib.h>

#include <map>
#include <set>
#include <thread>
#include <vector>

#include "../../paper_2608_10103_b200/csrc/workspace_pool.h"

struct FakeState {
  std::mutex m;
  int next_id = 1;
  std::set<void*> live;
  std::vector<std::pair<void*, int>> freed_after;  // (ptr, stream)
  std::map<int, bool> event_done;                  // event id -> done
  std::set<int> capturing;
  int allocs = 0, clears = 0, next_event = 1;
  bool queried_during_capture = false;
};

struct FakeBackend {
  using Stream = int;
  using Event = int;
  FakeState* st;
  int alloc(void** p, size_t bytes, Stream) {
    std::lock_guard<std::mutex> l(st->m);
    *p = malloc(bytes ? bytes : 1);
    st->live.insert(*p);
    ++st->allocs;
    return 0;
  }
  int free_after(void* p, Stream s) {
    std::lock_guard<std::mutex> l(st->m);
    st->freed_after.push_back({p, s});
    st->live.erase(p);
    return 0;
  }
  int free_now(void* p) {
    std::lock_guard<std::mutex> l(st->m);
    st->live.erase(p);
    free(p);
    return 0;
  }
  int event_create(Event* e) {
    std::lock_guard<std::mutex> l(st->m);
    *e = st->next_event++;
    st->event_done[*e] = true;  // never recorded = done
    return 0;
  }
  void event_destroy(Event) {}
  int event_record(Event e, Stream) {
    std::lock_guard<std::mutex> l(st->m);
    st->event_done[e] = false;  // the test marks completion by hand
    return 0;
  }
  bool event_done(Event e) {
    std::lock_guard<std::mutex> l(st->m);
    if (!st->capturing.empty()) st->queried_during_capture = true;  // not allowed in a capture
    return st->event_done[e];
  }
  bool capturing(Stream s) {
    std::lock_guard<std::mutex> l(st->m);
    return st->capturing.count(s) != 0;
  }
  int clear(void*, size_t, Stream) {
    std::lock_guard<std::mutex> l(st->m);
    ++st->clears;
    return 0;
  }
};

#define EXPECT(cond)                                             \
  do {                                                           \
    if (!(cond)) {                                               \
      printf("FAILED line %d: %s\n", __LINE__, #cond);           \
      return 1;                                                  \
    }                                                            \
  } while (0)

using Pool = b200gemm::WorkspacePool<FakeBackend>;

int main() {
  FakeState st;
  Pool pool(FakeBackend{&st});
  Pool::Lease a, b, c, d;

  // the same stream reuses its buffer; nothing new is allocated
  EXPECT(pool.acquire(1, 1000, 256, &a) == 0);
  EXPECT(st.allocs == 1 && st.clears == 1 && a.bytes >= 1000 && a.head_bytes >= 256);
  EXPECT(pool.release(a, 1) == 0);
  EXPECT(pool.acquire(1, 800, 256, &b) == 0);
  EXPECT(b.ptr == a.ptr && st.allocs == 1);
  EXPECT(pool.release(b, 1) == 0);

  // another stream does not get it while stream 1's work may still run ...
  EXPECT(pool.acquire(2, 500, 256, &c) == 0);
  EXPECT(c.ptr != a.ptr && st.allocs == 2 && pool.buffers() == 2);
  EXPECT(pool.release(c, 2) == 0);
  // ... but does once that work has completed
  for (auto& e : st.event_done) e.second = true;
  EXPECT(pool.acquire(3, 900, 256, &d) == 0);
  EXPECT(d.ptr == a.ptr && st.allocs == 2);
  EXPECT(pool.release(d, 3) == 0);

  // growth: stream 2's buffer is too small -> freed after stream 2's earlier work, new one
  // allocated, no third pool entry
  void* old_c = c.ptr;
  EXPECT(pool.acquire(2, 5000, 256, &c) == 0);
  EXPECT(st.allocs == 3 && pool.buffers() == 2 && c.bytes >= 5000);
  EXPECT(st.freed_after.size() == 1 && st.freed_after[0].first == old_c && st.freed_after[0].second == 2);
  // while stream 2's lease is out, a second thread on stream 2 gets a buffer of its own
  Pool::Lease c2;
  std::thread t([&] { pool.acquire(2, 100, 256, &c2); });
  t.join();
  EXPECT(c2.ptr != c.ptr);
  EXPECT(pool.release(c2, 2) == 0 && pool.release(c, 2) == 0);

  // a larger bookkeeping head than the buffer has: not reused as it is
  Pool::Lease h;
  const int before = st.allocs;
  EXPECT(pool.acquire(2, 100, 4096, &h) == 0);
  EXPECT(st.allocs == before + 1 && h.head_bytes >= 4096);
  EXPECT(pool.release(h, 2) == 0);

  // capture: nothing may be allocated; a fitting buffer is taken and stays shared
  st.capturing.insert(7);
  Pool::Lease g;
  const int allocs_before = st.allocs;
  EXPECT(pool.acquire(7, 1 << 30, 256, &g) == Pool::kNoAllocInCapture);
  EXPECT(pool.acquire(7, 4000, 256, &g) == 0);
  EXPECT(st.allocs == allocs_before);
  EXPECT(pool.release(g, 7) == 0);
  EXPECT(!st.queried_during_capture);
  // a shared buffer never moves to another stream through the "completed" rule
  for (auto& e : st.event_done) e.second = true;
  Pool::Lease k;
  st.capturing.clear();
  EXPECT(pool.acquire(9, 4000, 256, &k) == 0);
  EXPECT(k.ptr != g.ptr);
  EXPECT(pool.release(k, 9) == 0);

  // two threads with different streams, many rounds: never the same buffer at the same time
  std::vector<void*> seen[2];
  bool clash = false;
  std::mutex sm;
  std::set<void*> held;
  auto worker = [&](int stream, int idx) {
    for (int i = 0; i < 200; ++i) {
      Pool::Lease l;
      if (pool.acquire(stream, 300 + 50 * idx, 256, &l) != 0) { clash = true; return; }
      {
        std::lock_guard<std::mutex> g2(sm);
        if (!held.insert(l.ptr).second) clash = true;
        seen[idx].push_back(l.ptr);
      }
      std::this_thread::yield();
      {
        std::lock_guard<std::mutex> g2(sm);
        held.erase(l.ptr);
      }
      pool.release(l, stream);
    }
  };
  std::thread t1(worker, 11, 0), t2(worker, 12, 1);
  t1.join();
  t2.join();
  EXPECT(!clash);
  EXPECT(seen[0].front() != seen[1].front());

  // release_all frees what is not leased and keeps slots usable
  Pool::Lease z;
  EXPECT(pool.acquire(1, 10, 256, &z) == 0);
  EXPECT(pool.release_all() == 0);
  EXPECT(pool.buffers() == 1);
  EXPECT(pool.release(z, 1) == 0);
  EXPECT(pool.release_all() == 0 && pool.buffers() == 0);
  EXPECT(pool.acquire(1, 10, 256, &z) == 0 && pool.buffers() == 1);
  printf("ok\n");
  return 0;
}
