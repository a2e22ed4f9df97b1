// Library-owned device scratch memory, handed out per call so that calls on different streams
// never share it while either is in flight.
//
// Two kinds of scratch exist: the workspace of partial tiles (split-K, stream-K tail) and the
// buffer for packed or transposed copies of operands. A "lease" owns one of each. A call that
// needs scratch holds exactly one lease from its first request until its last kernel has been
// enqueued; the lease then remembers the stream and, once more than one stream is in play, an
// event recorded behind that last kernel. The next call may take a lease
//   1. that was last used on the same stream (stream order already serialises the two calls),
//   2. whose event has completed (or that was never used),
//   3. that is new (up to kMaxLeases per device: memory grows only with real concurrency),
//   4. or, failing all that, the least recently used one after making its own stream wait for
//      that lease's event.
// As long as every call on a device has come from one and the same stream no event is recorded
// at all (rule 1 always applies), so the single-stream path costs a mutex and a pointer compare.
// The first call from a second stream synchronises the device once and switches the pool to
// recording events from then on.
//
// Stream capture: no event is recorded or queried on a capturing stream and nothing is allocated
// (allocation would invalidate the capture): a captured call uses the lease of its stream, or
// the first lease, as it stands. Replays of such a graph are outside the guarantee above.
//
// Host only; plain CUDA runtime calls. Used by the FP64 and the FP32 halves of the library, each
// with a pool array of its own.
#pragma once

#include <cstddef>
#include <mutex>

#include <cuda_runtime.h>

namespace scratch {

constexpr int kMaxLeases = 4;

struct Lease {
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  void* pack = nullptr;
  size_t pack_bytes = 0;
  cudaEvent_t done = nullptr;       // behind the last kernel that used the lease (multi-stream mode only)
  bool recorded = false;            // `done` has been recorded at least once since the lease was last free for sure
  cudaStream_t last_stream = nullptr;
  bool used = false;
  unsigned long long tick = 0;      // order of last use
};

struct Pool {
  std::mutex mu;                    // held by a call from its first request to its last launch
  Lease lease[kMaxLeases];
  int count = 0;
  bool multi_stream = false;        // a second stream has been seen: events are recorded from now on
  cudaStream_t only_stream = nullptr;
  bool any_use = false;
  unsigned long long tick = 0;
};

enum Kind { kWorkspace = 0, kPack = 1 };

// One call's claim on a lease. Construct it before the first kernel of the call is launched and
// let it go out of scope after the last one: the destructor records the lease's event (when events
// are in use) and lets the next caller in.
class Hold {
 public:
  Hold(Pool& pool, cudaStream_t stream) : pool_(pool), stream_(stream) {}
  Hold(const Hold&) = delete;
  Hold& operator=(const Hold&) = delete;

  ~Hold() {
    if (!lease_) return;
    if (!capturing_) {
      if (pool_.multi_stream) {
        if (lease_->done && cudaEventRecord(lease_->done, stream_) == cudaSuccess) lease_->recorded = true;
        else (void)cudaGetLastError();
      }
      lease_->used = true;
      lease_->last_stream = stream_;
      lease_->tick = ++pool_.tick;
    }
    pool_.mu.unlock();
  }

  // At least `bytes` of device memory for partial tiles, or nullptr (allocation failed, or a first
  // use under stream capture). The contents are whatever the previous user left.
  void* workspace(size_t bytes) { return get(kWorkspace, bytes, 0); }

  // At least `bytes` for packed operands; grown with `bytes / 4` of head room against regrowing on
  // slightly larger problems.
  void* pack_buffer(size_t bytes) { return get(kPack, bytes, bytes / 4); }

 private:
  static bool satisfies(const Lease& l, Kind kind, size_t bytes) {
    return (kind == kWorkspace ? l.workspace_bytes : l.pack_bytes) >= bytes;
  }

  bool is_capturing() const {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream_, &cs) != cudaSuccess) {
      (void)cudaGetLastError();
      return false;
    }
    return cs != cudaStreamCaptureStatusNone;
  }

  Lease* new_lease() {
    if (pool_.count >= kMaxLeases) return nullptr;
    Lease& l = pool_.lease[pool_.count];
    l = Lease();
    ++pool_.count;
    return &l;
  }

  bool acquire(Kind kind, size_t bytes) {
    pool_.mu.lock();
    Lease* pick = nullptr;
    if (!pool_.multi_stream) {
      if (!pool_.any_use || stream_ == pool_.only_stream) {
        // (a first-ever call under capture will fail at its allocation, like any allocation under capture)
        pick = pool_.count > 0 ? &pool_.lease[0] : new_lease();
        if (!pool_.any_use) {
          pool_.any_use = true;
          pool_.only_stream = stream_;
        }
      } else if ((capturing_ = is_capturing())) {
        pick = pool_.count > 0 ? &pool_.lease[0] : new_lease();
      } else {
        // A second stream. Nothing has recorded events so far, so let everything issued up to now
        // finish, once, and start recording.
        if (cudaDeviceSynchronize() != cudaSuccess) {
          (void)cudaGetLastError();
          pool_.mu.unlock();
          return false;
        }
        pool_.multi_stream = true;
        for (int i = 0; i < pool_.count; ++i) {
          pool_.lease[i].used = false;
          pool_.lease[i].recorded = false;
        }
      }
    } else {
      capturing_ = is_capturing();
    }
    if (!pick && capturing_) {
      for (int i = 0; i < pool_.count && !pick; ++i)
        if (pool_.lease[i].used && pool_.lease[i].last_stream == stream_) pick = &pool_.lease[i];
      if (!pick && pool_.count > 0) pick = &pool_.lease[0];
    }
    if (!pick && pool_.multi_stream && !capturing_) {
      // rule 1: same stream
      for (int i = 0; i < pool_.count && !pick; ++i)
        if (pool_.lease[i].used && pool_.lease[i].last_stream == stream_) pick = &pool_.lease[i];
      // rule 2: finished or never used; one that already holds enough memory first
      if (!pick) {
        Lease* spare = nullptr;
        for (int i = 0; i < pool_.count; ++i) {
          Lease& l = pool_.lease[i];
          bool is_free = !l.used || !l.recorded;
          if (!is_free) {
            const cudaError_t q = cudaEventQuery(l.done);
            if (q == cudaSuccess) {
              is_free = true;
              l.used = false;  // nothing of its last user is in flight any more
            } else {
              (void)cudaGetLastError();  // "not ready" is also left behind as the last error: clear it
            }
          }
          if (!is_free) continue;
          if (satisfies(l, kind, bytes)) {
            pick = &l;
            break;
          }
          if (!spare) spare = &l;
        }
        if (!pick) pick = spare;
      }
      // rule 3: one more lease
      if (!pick) pick = new_lease();
      // rule 4: wait for the one used longest ago
      if (!pick) {
        for (int i = 0; i < pool_.count; ++i)
          if (!pick || pool_.lease[i].tick < pick->tick) pick = &pool_.lease[i];
        if (pick && cudaStreamWaitEvent(stream_, pick->done, 0) != cudaSuccess) {
          (void)cudaGetLastError();
          pick = nullptr;
        }
      }
    }
    if (pick && pool_.multi_stream && !capturing_ && !pick->done &&
        cudaEventCreateWithFlags(&pick->done, cudaEventDisableTiming) != cudaSuccess) {
      (void)cudaGetLastError();
      pick = nullptr;
    }
    if (!pick) {
      pool_.mu.unlock();
      return false;
    }
    lease_ = pick;
    return true;
  }

  void* get(Kind kind, size_t bytes, size_t head_room) {
    if (!lease_ && !acquire(kind, bytes)) return nullptr;
    void*& buf = kind == kWorkspace ? lease_->workspace : lease_->pack;
    size_t& have = kind == kWorkspace ? lease_->workspace_bytes : lease_->pack_bytes;
    if (have >= bytes) return buf;
    if (capturing_) return nullptr;  // growing means allocating, which a capture does not survive
    if (buf) {
      // the buffer being replaced may still be read by this stream's earlier kernels (no other
      // stream can hold this lease): let them finish before it is freed
      if (cudaStreamSynchronize(stream_) != cudaSuccess) (void)cudaGetLastError();
      cudaFree(buf);
      buf = nullptr;
      have = 0;
    }
    const size_t want = bytes + head_room;
    if (cudaMalloc(&buf, want) != cudaSuccess) {
      (void)cudaGetLastError();
      buf = nullptr;
      return nullptr;
    }
    have = want;
    return buf;
  }

  Pool& pool_;
  cudaStream_t stream_;
  Lease* lease_ = nullptr;
  bool capturing_ = false;
};

// Frees everything the pool holds and returns it to its initial single-stream state. The caller
// has synchronised the device. Returns false if a free failed.
inline bool release_all(Pool& pool) {
  std::lock_guard<std::mutex> lock(pool.mu);
  bool ok = true;
  for (int i = 0; i < pool.count; ++i) {
    Lease& l = pool.lease[i];
    if (l.workspace) ok = cudaFree(l.workspace) == cudaSuccess && ok;
    if (l.pack) ok = cudaFree(l.pack) == cudaSuccess && ok;
    if (l.done) ok = cudaEventDestroy(l.done) == cudaSuccess && ok;
    l = Lease();
  }
  pool.count = 0;
  pool.multi_stream = false;
  pool.any_use = false;
  pool.only_stream = nullptr;
  return ok;
}

}  // namespace scratch
