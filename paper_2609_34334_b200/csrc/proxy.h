// Stream manager in the paper's form (Sec. 3.2): a CPU proxy thread that takes over a GPU stream through a
// two-flag handshake carried by stream memory operations, runs the communication, and hands the stream back.
//
// Per operation the caller's stream gets four memory operations (Listing 1 of the paper, in our words):
//     write  start_flag  <- START          the stream tells the CPU it has reached the operation
//     wait   start_flag  == 0              the CPU has seen it (acknowledgement)
//     wait   finish_flag >= FINISH         the CPU reports that the communication is complete
//     write  finish_flag <- 0              the stream acknowledges, the flag pair can be reused
// The flags live in pinned host memory; the proxy polls them.  No SM is involved in the hand-over.
// Per flag pair the proxy walks a small state machine (the analogue of the paper's per-chunk buffer states):
//     FREE -> WAIT_START -> (PARKED for an unmatched send/recv) -> RUNNING -> WAIT_ACK -> FREE
// A watchdog bounds every state: after `watchdog_ms` the proxy releases the stream with the ABORT value (which the
// >= wait accepts) and records a sticky error, so a stream can never wait forever on this library.
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

constexpr uint32_t kFlagStart = 1;
constexpr uint32_t kFlagFinish = 1;
constexpr uint32_t kFlagAbort = 2;
constexpr int kFlagPairs = 64;

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
  // filled by the proxy
  int pair = -1;
};

enum ProxyError { PROXY_OK = 0, PROXY_TIMEOUT = 1, PROXY_MISMATCH = 2, PROXY_CUDA = 3 };

class Proxy {
 public:
  Proxy(int device, long watchdog_ms);
  ~Proxy();
  cudaError_t init();  // resolves the driver entry points, allocates the flag pool, starts the thread
  // Enqueues the four stream memory operations on `user` and hands the task to the thread.  Blocks only when all
  // flag pairs are in use (bounded by the watchdog).  Returns cudaErrorUnknown if the proxy has been shut down.
  cudaError_t submit(cudaStream_t user, ProxyTask task);
  int pending_p2p();           // send/recv posts parked without a partner
  int async_error();           // sticky ProxyError of the first failure
  void clear_error();
  bool drain(long timeout_ms); // waits until no task is active
  void set_watchdog_ms(long ms) { watchdog_ms_ = ms; }
  long handshakes() const { return handshakes_.load(); }
  cudaStream_t work_stream() const { return stream_; }

 private:
  enum State { FREE = 0, WAIT_START, READY, PARKED, RUNNING, WAIT_ACK };
  struct Slot {
    State state = FREE;
    ProxyTask task;
    double t0 = 0;
    cudaEvent_t done = nullptr;
    int partner = -1;  // P2P: the other slot of a matched pair
  };
  void loop();
  void release_with_abort(int i, int err);
  volatile uint32_t* start_flag(int i) { return flags_ + 2 * i; }
  volatile uint32_t* finish_flag(int i) { return flags_ + 2 * i + 1; }

  int device_;
  std::atomic<long> watchdog_ms_;
  volatile uint32_t* flags_ = nullptr;  // pinned host memory, 2 words per pair
  uint32_t* flags_dev_ = nullptr;       // the same memory as the device sees it
  void* fn_write_ = nullptr;
  void* fn_wait_ = nullptr;
  cudaStream_t stream_ = nullptr;
  void* warm_ = nullptr;  // 512 bytes of device memory used once, to exercise the copy route before any hand-over
  std::thread th_;
  std::mutex mu_;
  std::condition_variable cv_;
  std::deque<ProxyTask> inbox_;
  std::vector<Slot> slots_;
  std::atomic<int> active_{0};
  std::atomic<int> parked_{0};
  std::atomic<int> error_{0};
  std::atomic<long> handshakes_{0};
  std::atomic<bool> stop_{false};
  int next_pair_ = 0;
  std::vector<char> pair_busy_;  // guarded by mu_
};

}  // namespace hoccl
