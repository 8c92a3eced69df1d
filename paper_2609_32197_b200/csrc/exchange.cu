// Transfer runtime of the demand-routed exchange (Section 6): reusable peer-visible slots and the five
// primitives Export / Publish / Fetch / Release / Fence, plus the per-hop pack of one (consumer, producer)
// segment into a slot.
//
// B200 form of the paper's design:
//   * a rank's slot window is plain device memory that its peers can address (on one device: any device
//     pointer; across GPUs of a node: a peer mapping the caller obtained and registers with
//     sparsp_xchg_connect); every slot has the same size on every rank (Section 6.2: same geometry
//     everywhere, so a consumer derives every byte range locally);
//   * Fetch is ONE asynchronous copy per planned transfer on the consumer's copy stream -- the copy engines
//     move the bytes over NVLink, no SM takes part (Section 6.2), and the payload lands in the consumer's own
//     memory before any kernel (or TMA load) touches it;
//   * Publish and Release are 4-byte sequence numbers in a flag page every rank can read and write from the
//     HOST (pinned or inter-process shared memory).  They are stored by a host function enqueued on the
//     stream that produced the data (pack stream for Publish, copy stream for Release), so stream order
//     gives "payload complete before notification" (Section 6.1) without a kernel;
//   * every wait (a producer waiting for a slot to be released, a consumer waiting for a publication) is a
//     HOST-side poll with a time limit: it returns SPARSP_ERR_TIMEOUT, never blocks for ever, and no kernel
//     ever spins on another rank;
//   * Fence separates attention calls: the caller's barrier (NCCL / gloo / a thread barrier for virtual
//     ranks) followed by sparsp_xchg_fence, which moves the endpoint to the next epoch; sequence numbers carry
//     the epoch, so flags of an earlier call can never satisfy a wait of a later one.
// A host-memory mode (slots in host memory, copies by memcpy, flag stores done at once) exists so that the
// slot state machine can be exercised by multi-process tests on machines without a GPU.
#include <time.h>

#include <atomic>
#include <cstring>
#include <new>

#include "common.cuh"

namespace sparsp {

constexpr int kXchgMaxWindow = 64;

// one int32 pair per (rank, slot): [0] = sequence number of the latest publication, [1] = of the latest release
static inline int64_t flag_index(int window, int rank, int slot, int which) {
  return ((int64_t)rank * window + slot) * 2 + which;
}

static inline int32_t seq_of(int32_t epoch, int64_t use) { return (int32_t)((epoch & 0x7fff) << 16) | (int32_t)((use & 0xffff) + 1); }

static inline int64_t now_us() {
  timespec ts;
  clock_gettime(CLOCK_MONOTONIC, &ts);
  return (int64_t)ts.tv_sec * 1000000 + ts.tv_nsec / 1000;
}

struct FlagStore {
  int32_t* addr;
  int32_t value;
};

static void CUDART_CB flag_store_cb(void* p) {
  FlagStore* f = static_cast<FlagStore*>(p);
  __atomic_store_n(f->addr, f->value, __ATOMIC_RELEASE);
  delete f;
}

}  // namespace sparsp

struct sparsp_xchg {
  int32_t P, rank, window, host_memory, epoch;
  int64_t slot_bytes, wait_limit_us;
  char* slots;
  char* peer_slots[sparsp::kMaxRanks];
  int32_t* flags;
  // statistics: publications, fetches, releases, acquisitions that had to wait, bytes fetched, microseconds
  // spent waiting for a release / for a publication, timeouts
  std::atomic<int64_t> stats[8];
};

using namespace sparsp;

// Polls *addr until it equals `want` or the endpoint's time limit runs out.
static int wait_flag(sparsp_xchg* x, int32_t* addr, int32_t want, const char* what, int who, int slot, int stat) {
  if (__atomic_load_n(addr, __ATOMIC_ACQUIRE) == want) return SPARSP_OK;
  const int64_t t0 = now_us();
  int spins = 0;
  for (;;) {
    if (__atomic_load_n(addr, __ATOMIC_ACQUIRE) == want) {
      x->stats[stat].fetch_add(now_us() - t0);
      return SPARSP_OK;
    }
    if (++spins > 64) {
      timespec nap = {0, 20000};  // 20 us: the waits here are for GPU work of hundreds of microseconds
      nanosleep(&nap, nullptr);
    }
    if (now_us() - t0 > x->wait_limit_us) {
      x->stats[stat].fetch_add(now_us() - t0);
      x->stats[7].fetch_add(1);
      if (who == x->rank)
        set_error("rank %d: waited %lld us for the consumer of its slot %d to %s it (flag %d, wanted %d)", x->rank,
                  (long long)x->wait_limit_us, slot, what, __atomic_load_n(addr, __ATOMIC_ACQUIRE), want);
      else
        set_error("rank %d: waited %lld us for rank %d to %s slot %d (flag %d, wanted %d)", x->rank,
                  (long long)x->wait_limit_us, who, what, slot, __atomic_load_n(addr, __ATOMIC_ACQUIRE), want);
      return SPARSP_ERR_TIMEOUT;
    }
  }
}

static int store_flag(sparsp_xchg* x, int32_t* addr, int32_t value, void* stream) {
  if (x->host_memory) {
    __atomic_store_n(addr, value, __ATOMIC_RELEASE);
    return SPARSP_OK;
  }
  FlagStore* f = new (std::nothrow) FlagStore{addr, value};
  if (!f) {
    set_error("out of host memory");
    return SPARSP_ERR_CUDA;
  }
  cudaError_t e = cudaLaunchHostFunc((cudaStream_t)stream, flag_store_cb, f);
  if (e != cudaSuccess) {
    delete f;
    return cuda_fail(e, "cudaLaunchHostFunc");
  }
  return SPARSP_OK;
}

#define XCHG_CHECK(x)                     \
  do {                                    \
    if (!(x)) {                           \
      set_error("exchange handle is NULL"); \
      return SPARSP_ERR_INVALID_ARG;      \
    }                                     \
  } while (0)

extern "C" {

int sparsp_xchg_flag_bytes(int32_t n_ranks, int32_t window, int64_t* bytes) {
  if (n_ranks < 1 || n_ranks > kMaxRanks || window < 1 || window > kXchgMaxWindow || !bytes) {
    set_error("n_ranks %d outside 1..%d, window %d outside 1..%d, or NULL output", n_ranks, kMaxRanks, window,
              kXchgMaxWindow);
    return SPARSP_ERR_INVALID_ARG;
  }
  *bytes = (int64_t)n_ranks * window * 2 * 4;
  return SPARSP_OK;
}

int sparsp_xchg_export(int32_t n_ranks, int32_t rank, int32_t window, int64_t slot_bytes, void* slots,
                       void* flag_page, int64_t wait_limit_us, int32_t flags, sparsp_xchg** out) {
  int64_t fb = 0;
  int rc = sparsp_xchg_flag_bytes(n_ranks, window, &fb);
  if (rc != SPARSP_OK) return rc;
  if (rank < 0 || rank >= n_ranks || slot_bytes < 16 || slot_bytes % 16 || !slots || (uintptr_t)slots % 16 ||
      !flag_page || (uintptr_t)flag_page % 4 || wait_limit_us < 1 || !out || (flags & ~SPARSP_XCHG_HOST_MEMORY)) {
    set_error("bad rank, slot size (a positive multiple of 16), pointer, time limit or flag bits");
    return SPARSP_ERR_INVALID_ARG;
  }
  sparsp_xchg* x = new (std::nothrow) sparsp_xchg;
  if (!x) {
    set_error("out of host memory");
    return SPARSP_ERR_CUDA;
  }
  x->P = n_ranks;
  x->rank = rank;
  x->window = window;
  x->host_memory = (flags & SPARSP_XCHG_HOST_MEMORY) ? 1 : 0;
  x->epoch = 1;
  x->slot_bytes = slot_bytes;
  x->wait_limit_us = wait_limit_us;
  x->slots = (char*)slots;
  for (int r = 0; r < kMaxRanks; ++r) x->peer_slots[r] = nullptr;
  x->peer_slots[rank] = (char*)slots;
  x->flags = (int32_t*)flag_page;
  for (auto& s : x->stats) s.store(0);
  *out = x;
  return SPARSP_OK;
}

int sparsp_xchg_connect(sparsp_xchg* x, int32_t peer, void* peer_slots) {
  XCHG_CHECK(x);
  if (peer < 0 || peer >= x->P || !peer_slots || (uintptr_t)peer_slots % 16) {
    set_error("peer %d outside 0..%d or bad window address", peer, x->P - 1);
    return SPARSP_ERR_INVALID_ARG;
  }
  x->peer_slots[peer] = (char*)peer_slots;
  return SPARSP_OK;
}

int sparsp_xchg_fence(sparsp_xchg* x) {
  XCHG_CHECK(x);
  x->epoch = (x->epoch % 0x7fff) + 1;
  return SPARSP_OK;
}

int sparsp_xchg_acquire(sparsp_xchg* x, int64_t use, int32_t* slot, void** slot_ptr) {
  XCHG_CHECK(x);
  if (use < 0 || use > 0xfffe || !slot) {
    set_error("use %lld outside 0..65534 or NULL output", (long long)use);
    return SPARSP_ERR_INVALID_ARG;
  }
  const int s = (int)(use % x->window);
  if (use >= x->window) {
    // the slot's previous content (use - window of this call) must have been released by its consumer
    int32_t* rel = x->flags + flag_index(x->window, x->rank, s, 1);
    const bool free_now = __atomic_load_n(rel, __ATOMIC_ACQUIRE) == seq_of(x->epoch, use - x->window);
    if (!free_now) x->stats[3].fetch_add(1);
    int rc = wait_flag(x, rel, seq_of(x->epoch, use - x->window), "release", x->rank, s, 5);
    if (rc != SPARSP_OK) return rc;
  }
  *slot = s;
  if (slot_ptr) *slot_ptr = x->slots + (int64_t)s * x->slot_bytes;
  return SPARSP_OK;
}

int sparsp_xchg_publish(sparsp_xchg* x, int64_t use, void* stream) {
  XCHG_CHECK(x);
  if (use < 0 || use > 0xfffe) {
    set_error("use %lld outside 0..65534", (long long)use);
    return SPARSP_ERR_INVALID_ARG;
  }
  const int s = (int)(use % x->window);
  x->stats[0].fetch_add(1);
  return store_flag(x, x->flags + flag_index(x->window, x->rank, s, 0), seq_of(x->epoch, use), stream);
}

int sparsp_xchg_fetch(sparsp_xchg* x, int32_t producer, int64_t use, int64_t src_offset, void* dst, int64_t n_bytes,
                      void* copy_stream) {
  XCHG_CHECK(x);
  if (producer < 0 || producer >= x->P || producer == x->rank || use < 0 || use > 0xfffe || src_offset < 0 ||
      n_bytes < 0 || src_offset + n_bytes > x->slot_bytes || (n_bytes > 0 && !dst)) {
    set_error("bad producer %d, use %lld, or byte range [%lld, +%lld) outside a slot of %lld bytes", producer,
              (long long)use, (long long)src_offset, (long long)n_bytes, (long long)x->slot_bytes);
    return SPARSP_ERR_INVALID_ARG;
  }
  if (!x->peer_slots[producer]) {
    set_error("rank %d: the slot window of rank %d has not been connected", x->rank, producer);
    return SPARSP_ERR_INVALID_ARG;
  }
  const int s = (int)(use % x->window);
  int rc = wait_flag(x, x->flags + flag_index(x->window, producer, s, 0), seq_of(x->epoch, use), "publish", producer,
                     s, 6);
  if (rc != SPARSP_OK) return rc;
  x->stats[1].fetch_add(1);
  x->stats[4].fetch_add(n_bytes);
  if (n_bytes == 0) return SPARSP_OK;
  const char* src = x->peer_slots[producer] + (int64_t)s * x->slot_bytes + src_offset;
  if (x->host_memory) {
    memcpy(dst, src, (size_t)n_bytes);
    return SPARSP_OK;
  }
  // one copy per planned transfer; between two devices of a node the runtime routes it over NVLink
  SPARSP_CUDA_OK(cudaMemcpyAsync(dst, src, (size_t)n_bytes, cudaMemcpyDefault, (cudaStream_t)copy_stream));
  return SPARSP_OK;
}

int sparsp_xchg_release(sparsp_xchg* x, int32_t producer, int64_t use, void* copy_stream) {
  XCHG_CHECK(x);
  if (producer < 0 || producer >= x->P || producer == x->rank || use < 0 || use > 0xfffe) {
    set_error("bad producer %d or use %lld", producer, (long long)use);
    return SPARSP_ERR_INVALID_ARG;
  }
  const int s = (int)(use % x->window);
  x->stats[2].fetch_add(1);
  return store_flag(x, x->flags + flag_index(x->window, producer, s, 1), seq_of(x->epoch, use), copy_stream);
}

int sparsp_xchg_stats(sparsp_xchg* x, int64_t* out) {
  XCHG_CHECK(x);
  if (!out) {
    set_error("out is NULL");
    return SPARSP_ERR_INVALID_ARG;
  }
  for (int i = 0; i < 8; ++i) out[i] = x->stats[i].load();
  return SPARSP_OK;
}

int sparsp_xchg_destroy(sparsp_xchg* x) {
  XCHG_CHECK(x);
  delete x;
  return SPARSP_OK;
}

}  // extern "C"
