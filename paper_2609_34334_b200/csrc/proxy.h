// Stream manager with a CPU proxy thread (the idea of the paper's Sec. 3.2: a GPU stream hands itself to a CPU thread
// through flags that stream memory operations write and wait on, the CPU drives the communication, and the stream goes
// on when the CPU says so).  The hand-over protocol here is this library's own: sequence numbered, no flag is ever reset.
//
// Every flag pair i has three 32-bit counters in pinned host memory that only grow:
//     arrived[i]   written by the GPU stream: "hand-over number n has reached this point of the stream"
//     released[i]  written by the proxy:      "hand-over number n may go on"
//     passed[i]    written by the GPU stream: "hand-over number n is behind me"
// One hand-over with number n on pair i is three stream memory operations on the caller's stream:
//     write arrived[i] <- n;   wait released[i] >= n (cyclic compare);   write passed[i] <- n
// and on the proxy's side: see arrived[i] == n, run the work on the proxy's own stream, see it finish, write
// released[i] <- n.  Because the counters only grow, nothing has to be acknowledged or reset before a pair is used
// again, and a stream can be let go at ANY time, even before it has arrived, by writing released[i] <- n: that is how
// the watchdog (an unmatched send/recv, work that does not finish) and the shutdown release streams, so no stream can
// wait on this library forever.  `passed` only tells the host when the flag memory is no longer needed.
// Per pair the proxy walks a small state machine: FREE -> WAIT_ARRIVE -> READY -> (PARKED, an unmatched send/recv) ->
// RUNNING -> FREE.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <condition_variable>
#include <cstdint>
#include <deque>
#include <mutex>
#include <thread>
#include <vector>

namespace hoccl {

constexpr int kFlagPairs = 64;
constexpr int kFlagWords = 4;  // arrived, released, passed, (unused): one pair per 16 bytes

struct ProxyTask {
  enum Kind { GRAPH = 0, P2P = 1 };
  int kind = GRAPH;
  cudaGraphExec_t exec = nullptr;  // GRAPH: what to launch on the proxy's stream
  // P2P
  bool is_send = false;
  int src = 0, dst = 0;
  void* buf = nullptr;
  size_t count = 0, elem = 0;
  int dtype = 0;
  int path = 0, copy_ctas = 8;
  // filled by submit
  int pair = -1;
  uint32_t seq = 0;
};

enum ProxyError { PROXY_OK = 0, PROXY_TIMEOUT = 1, PROXY_MISMATCH = 2, PROXY_CUDA = 3 };

class Proxy {
 public:
  Proxy(int device, long watchdog_ms);
  ~Proxy();
  cudaError_t init();  // resolves the driver entry points, allocates the flag pool, starts the thread
  // Enqueues the three stream memory operations on `user` and hands the task to the thread.  Blocks only when all
  // flag pairs are in use (bounded by the watchdog).  Returns cudaErrorUnknown if the proxy has been shut down.
  cudaError_t submit(cudaStream_t user, ProxyTask task);
  int pending_p2p();           // send/recv posts parked without a partner
  int async_error();           // sticky ProxyError of the first failure
  void clear_error();
  bool drain(long timeout_ms); // waits until no task is active (parked send/recv posts do not count)
  // Stops the thread.  Every hand-over that is still open is released first (its stream goes on, TIMEOUT is recorded),
  // then the call waits up to `timeout_ms` for every stream to get past its hand-over.  Returns true if all did: the
  // flag memory is freed by the destructor then.  false: some stream has not reached its hand-over yet; the flag
  // memory is kept for the life of the process (a few hundred bytes), so that stream still finds released[i] when it
  // gets there.
  bool shutdown(long timeout_ms);
  void set_watchdog_ms(long ms) { watchdog_ms_ = ms; }
  long handshakes() const { return handshakes_.load(); }
  // Time the thread spent working (launching schedules and moves, writing flags) and the wall time between the first
  // task it accepted and the last release, in microseconds: 1 - busy / span is the share of that time the thread only
  // polled (the analogue of the CPU slack the paper reports for its proxy, Sec. 5 "End-to-end workloads").
  void work_stats(double* busy_us, double* span_us) const;
  void reset_work_stats();
  cudaStream_t work_stream() const { return stream_; }

 private:
  enum State { FREE = 0, WAIT_ARRIVE, READY, PARKED, RUNNING };
  struct Slot {
    State state = FREE;
    ProxyTask task;
    double t0 = 0;
    cudaEvent_t done = nullptr;
    int partner = -1;  // P2P: the other slot of a matched pair
  };
  void loop();
  void release(int i, int err);   // lets the stream of slot i go on and frees the pair
  volatile uint32_t* arrived(int i) { return flags_ + kFlagWords * i; }
  volatile uint32_t* released(int i) { return flags_ + kFlagWords * i + 1; }
  volatile uint32_t* passed(int i) { return flags_ + kFlagWords * i + 2; }
  bool all_passed();

  int device_;
  std::atomic<long> watchdog_ms_;
  volatile uint32_t* flags_ = nullptr;  // pinned host memory, kFlagWords words per pair
  uint32_t* flags_dev_ = nullptr;       // the same memory as the device sees it
  bool keep_flags_ = false;             // shutdown could not see every stream pass: the flag memory must outlive us
  void* fn_write_ = nullptr;
  void* fn_wait_ = nullptr;
  cudaStream_t stream_ = nullptr;
  void* warm_ = nullptr;  // 512 bytes of device memory used once, to exercise the copy route before any hand-over
  std::thread th_;
  std::mutex mu_;
  std::condition_variable cv_;
  std::deque<ProxyTask> inbox_;
  std::vector<Slot> slots_;
  std::vector<uint32_t> last_seq_;   // per pair: the number of the latest hand-over enqueued on it (guarded by mu_)
  std::atomic<int> active_{0};
  std::atomic<int> parked_{0};
  std::atomic<int> error_{0};
  std::atomic<long> handshakes_{0};
  std::atomic<bool> stop_{false};
  std::atomic<long long> busy_ns_{0};
  std::atomic<long long> first_ns_{0}, last_ns_{0};
  int next_pair_ = 0;
  std::vector<char> pair_busy_;  // guarded by mu_
};

}  // namespace hoccl
