// CPU proxy thread and the sequence-numbered stream hand-over (see proxy.h; the idea of a stream that hands itself to a
// CPU thread is the paper's, Sec. 3.2; Sec. 3.3.2 for the matched send/recv that the proxy completes once both sides
// have posted).
#include "proxy.h"

#include <cuda.h>

#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstdlib>

#include "kernels.cuh"

namespace hoccl {

namespace {

typedef CUresult (*WriteValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
typedef CUresult (*WaitValue32Fn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);

bool trace_on() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("HOCCL_PROXY_TRACE");
    v = (e && e[0] == '1') ? 1 : 0;
  }
  return v == 1;
}
#define PTRACE(...)                      \
  do {                                   \
    if (trace_on()) {                    \
      fprintf(stderr, "[hoccl proxy] "); \
      fprintf(stderr, __VA_ARGS__);      \
      fprintf(stderr, "\n");             \
    }                                    \
  } while (0)

double now_ms() {
  return std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now().time_since_epoch()).count();
}
long long now_ns() {
  return std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

}  // namespace

Proxy::Proxy(int device, long watchdog_ms) : device_(device), watchdog_ms_(watchdog_ms) {
  slots_.resize(kFlagPairs);
  pair_busy_.assign(kFlagPairs, 0);
  last_seq_.assign(kFlagPairs, 0);
}

cudaError_t Proxy::init() {
  cudaError_t e = cudaSetDevice(device_);
  if (e != cudaSuccess) return e;
  cudaDriverEntryPointQueryResult qr;
  e = cudaGetDriverEntryPoint("cuStreamWriteValue32", &fn_write_, cudaEnableDefault, &qr);
  if (e != cudaSuccess || !fn_write_) return e != cudaSuccess ? e : cudaErrorNotSupported;
  e = cudaGetDriverEntryPoint("cuStreamWaitValue32", &fn_wait_, cudaEnableDefault, &qr);
  if (e != cudaSuccess || !fn_wait_) return e != cudaSuccess ? e : cudaErrorNotSupported;
  void* host = nullptr;
  e = cudaHostAlloc(&host, sizeof(uint32_t) * kFlagWords * kFlagPairs, cudaHostAllocMapped | cudaHostAllocPortable);
  if (e != cudaSuccess) return e;
  flags_ = static_cast<volatile uint32_t*>(host);
  for (int i = 0; i < kFlagWords * kFlagPairs; i++) flags_[i] = 0;
  void* dev = nullptr;
  e = cudaHostGetDevicePointer(&dev, host, 0);
  if (e != cudaSuccess) return e;
  flags_dev_ = static_cast<uint32_t*>(dev);
  e = cudaStreamCreateWithFlags(&stream_, cudaStreamNonBlocking);
  if (e != cudaSuccess) return e;
  for (auto& s : slots_) {
    e = cudaEventCreateWithFlags(&s.done, cudaEventDisableTiming);
    if (e != cudaSuccess) return e;
  }
  // Everything the proxy thread will ever launch is loaded and exercised once NOW, while no stream is parked:
  // first-use work inside the driver (kernel loading, the copy route, graph launch) may synchronise the device, and
  // a parked stream can only be released by this very thread.
  e = preload_kernels();
  if (e != cudaSuccess) return e;
  e = cudaMalloc(&warm_, 512);
  if (e != cudaSuccess) return e;
  e = cudaMemsetAsync(warm_, 0, 512, stream_);
  if (e == cudaSuccess) e = cudaMemcpyAsync(static_cast<char*>(warm_) + 256, warm_, 256, cudaMemcpyDeviceToDevice, stream_);
  if (e == cudaSuccess) {
    CopyBatch b;
    b.nseg = 1;
    b.pad = 0;
    b.seg[0] = CopySeg{warm_, static_cast<char*>(warm_) + 256, 256};
    e = launch_copy(b, 1, stream_);
  }
  cudaGraph_t g = nullptr;
  cudaGraphExec_t ge = nullptr;
  cudaGraphNode_t n;
  if (e == cudaSuccess) e = cudaGraphCreate(&g, 0);
  if (e == cudaSuccess) e = cudaGraphAddMemcpyNode1D(&n, g, nullptr, 0, static_cast<char*>(warm_) + 256, warm_, 256, cudaMemcpyDeviceToDevice);
  if (e == cudaSuccess) e = cudaGraphInstantiate(&ge, g, 0);
  if (e == cudaSuccess) e = cudaGraphLaunch(ge, stream_);
  if (e == cudaSuccess) e = cudaEventRecord(slots_[0].done, stream_);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream_);
  if (e == cudaSuccess) e = cudaEventQuery(slots_[0].done);
  if (ge) cudaGraphExecDestroy(ge);
  if (g) cudaGraphDestroy(g);
  if (e != cudaSuccess) return e;
  th_ = std::thread([this] { loop(); });
  return cudaSuccess;
}

bool Proxy::all_passed() {
  std::lock_guard<std::mutex> lock(mu_);
  for (int i = 0; i < kFlagPairs; i++)
    if (*passed(i) != last_seq_[i]) return false;
  return true;
}

bool Proxy::shutdown(long timeout_ms) {
  stop_ = true;
  cv_.notify_all();
  if (th_.joinable()) th_.join();   // the loop releases whatever is still open before it ends
  if (!flags_) return true;
  if (keep_flags_) return false;
  const double t0 = now_ms();
  while (!all_passed()) {
    if (now_ms() - t0 > (double)timeout_ms) {
      keep_flags_ = true;   // a stream will still come and look at its pair: the counters stay where they are
      return false;
    }
    std::this_thread::sleep_for(std::chrono::microseconds(100));
  }
  return true;
}

Proxy::~Proxy() {
  shutdown(2 * watchdog_ms_.load() + 100);
  cudaSetDevice(device_);
  if (stream_) {
    cudaStreamSynchronize(stream_);
    cudaStreamDestroy(stream_);
  }
  for (auto& s : slots_)
    if (s.done) cudaEventDestroy(s.done);
  if (flags_ && !keep_flags_) cudaFreeHost(const_cast<uint32_t*>(flags_));
  if (warm_) cudaFree(warm_);
}

cudaError_t Proxy::submit(cudaStream_t user, ProxyTask task) {
  if (stop_) return cudaErrorUnknown;
  int pair = -1;
  uint32_t seq = 0;
  {
    std::unique_lock<std::mutex> lock(mu_);
    const double t0 = now_ms();
    for (;;) {
      for (int k = 0; k < kFlagPairs; k++) {
        int i = (next_pair_ + k) % kFlagPairs;
        if (!pair_busy_[i]) {
          pair = i;
          break;
        }
      }
      if (pair >= 0) break;
      if (now_ms() - t0 > (double)watchdog_ms_) return cudaErrorTimeout;
      cv_.wait_for(lock, std::chrono::milliseconds(1));
    }
    pair_busy_[pair] = 1;
    next_pair_ = (pair + 1) % kFlagPairs;
    seq = ++last_seq_[pair];
  }
  const CUdeviceptr d_arrived = (CUdeviceptr)(uintptr_t)(flags_dev_ + kFlagWords * pair);
  const CUdeviceptr d_released = d_arrived + 4, d_passed = d_arrived + 8;
  WriteValue32Fn wr = reinterpret_cast<WriteValue32Fn>(fn_write_);
  WaitValue32Fn wt = reinterpret_cast<WaitValue32Fn>(fn_wait_);
  CUstream cs = (CUstream)user;
  // arrive, wait for the release of this very hand-over (cyclic >=, so the counters may wrap), tell the host we are past it
  CUresult r = wr(cs, d_arrived, seq, CU_STREAM_WRITE_VALUE_DEFAULT);
  if (r == CUDA_SUCCESS) r = wt(cs, d_released, seq, CU_STREAM_WAIT_VALUE_GEQ);
  if (r == CUDA_SUCCESS) r = wr(cs, d_passed, seq, CU_STREAM_WRITE_VALUE_DEFAULT);
  if (r != CUDA_SUCCESS) {
    // Whatever part was enqueued still has to be served: hand the proxy a task that does no work and is released at once.
    task.kind = ProxyTask::GRAPH;
    task.exec = nullptr;
    *passed(pair) = seq;   // nothing on the stream will write it
  }
  task.pair = pair;
  task.seq = seq;
  {
    std::lock_guard<std::mutex> lock(mu_);
    inbox_.push_back(task);
    active_++;
  }
  cv_.notify_all();
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorUnknown;
}

int Proxy::pending_p2p() { return parked_.load(); }
int Proxy::async_error() { return error_.load(); }
void Proxy::clear_error() { error_ = 0; }

void Proxy::work_stats(double* busy_us, double* span_us) const {
  if (busy_us) *busy_us = (double)busy_ns_.load() / 1e3;
  const long long a = first_ns_.load(), b = last_ns_.load();
  if (span_us) *span_us = (a && b > a) ? (double)(b - a) / 1e3 : 0.0;
}
void Proxy::reset_work_stats() {
  busy_ns_ = 0;
  first_ns_ = 0;
  last_ns_ = 0;
}

bool Proxy::drain(long timeout_ms) {
  const double t0 = now_ms();
  while (active_.load() > parked_.load()) {
    if (now_ms() - t0 > (double)timeout_ms) return false;
    std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
  return true;
}

// The stream of slot i may go on (err != PROXY_OK: it is let go without its result, and the first such error sticks).
void Proxy::release(int i, int err) {
  if (err != PROXY_OK) {
    int zero = 0;
    error_.compare_exchange_strong(zero, err);
  }
  std::atomic_thread_fence(std::memory_order_seq_cst);
  *released(i) = slots_[i].task.seq;
  std::atomic_thread_fence(std::memory_order_seq_cst);
  slots_[i].state = FREE;
  last_ns_ = now_ns();
  {
    std::lock_guard<std::mutex> lock(mu_);
    pair_busy_[i] = 0;
    active_--;
  }
  cv_.notify_all();
  PTRACE("pair %d: hand-over %u released (%d)", i, slots_[i].task.seq, err);
}

void Proxy::loop() {
  cudaSetDevice(device_);
  long seq = 0;
  std::vector<long> order(kFlagPairs, 0);  // arrival order of the task in each slot (FIFO matching)
  double stop_since = 0;
  for (;;) {
    {
      std::unique_lock<std::mutex> lock(mu_);
      while (!inbox_.empty()) {
        ProxyTask t = inbox_.front();
        inbox_.pop_front();
        Slot& s = slots_[t.pair];
        s.task = t;
        // a task without work comes from a hand-over that could not be enqueued completely: nothing may arrive, release it
        s.state = (t.kind == ProxyTask::GRAPH && !t.exec) ? READY : WAIT_ARRIVE;
        s.t0 = now_ms();
        s.partner = -1;
        order[t.pair] = seq++;
        if (first_ns_.load() == 0) first_ns_ = now_ns();
        PTRACE("pair %d: task kind %d accepted as hand-over %u", t.pair, t.kind, t.seq);
      }
      if (active_.load() == 0) {
        if (stop_) break;
        cv_.wait_for(lock, std::chrono::milliseconds(20));
        continue;
      }
    }
    if (stop_) {
      // Shutting down with hand-overs still open: they are served for at most one watchdog period; then every stream
      // that is still held, or has not even arrived yet, is let go (it finds its release whenever it gets there).
      if (stop_since == 0) stop_since = now_ms();
      if (now_ms() - stop_since > (double)watchdog_ms_) {
        for (int i = 0; i < kFlagPairs; i++)
          if (slots_[i].state != FREE) {
            if (slots_[i].state == PARKED) parked_--;
            release(i, PROXY_TIMEOUT);
          }
        break;
      }
    }
    const double now = now_ms();
    const double limit = (double)watchdog_ms_;
    std::this_thread::yield();
    for (int i = 0; i < kFlagPairs; i++) {
      Slot& s = slots_[i];
      switch (s.state) {
        case FREE:
          break;
        case WAIT_ARRIVE:
          if (*arrived(i) == s.task.seq) {
            std::atomic_thread_fence(std::memory_order_seq_cst);
            handshakes_++;
            PTRACE("pair %d: the stream has arrived", i);
            s.state = READY;
            s.t0 = now;
          } else if (now - s.t0 > limit) {
            int zero = 0;
            error_.compare_exchange_strong(zero, PROXY_TIMEOUT);  // reported, but the hand-over is still served
          }
          break;
        case READY: {
          const long long w0 = now_ns();
          if (s.task.kind == ProxyTask::GRAPH) {
            cudaError_t e = cudaSuccess;
            if (s.task.exec) e = cudaGraphLaunch(s.task.exec, stream_);
            if (e == cudaSuccess) e = cudaEventRecord(s.done, stream_);
            PTRACE("pair %d: schedule launched on the proxy stream (%s)", i, cudaGetErrorString(e));
            if (e != cudaSuccess) {
              release(i, PROXY_CUDA);
            } else {
              s.state = RUNNING;
              s.t0 = now;
            }
            busy_ns_ += now_ns() - w0;
            break;
          }
          // send/recv: look for the oldest parked partner of the same (src, dst) pair and the other direction
          int best = -1;
          for (int j = 0; j < kFlagPairs; j++) {
            const Slot& o = slots_[j];
            if (j != i && o.state == PARKED && o.task.src == s.task.src && o.task.dst == s.task.dst && o.task.is_send != s.task.is_send &&
                (best < 0 || order[j] < order[best]))
              best = j;
          }
          if (best < 0) {
            s.state = PARKED;
            s.t0 = now;
            parked_++;
            busy_ns_ += now_ns() - w0;
            break;
          }
          Slot& o = slots_[best];
          parked_--;
          if (o.task.count != s.task.count || o.task.dtype != s.task.dtype) {
            release(best, PROXY_MISMATCH);
            release(i, PROXY_MISMATCH);
            busy_ns_ += now_ns() - w0;
            break;
          }
          const void* src = s.task.is_send ? s.task.buf : o.task.buf;
          void* dst = s.task.is_send ? o.task.buf : s.task.buf;
          const size_t bytes = s.task.count * s.task.elem;
          cudaError_t e = cudaSuccess;
          if (bytes) {
            if (s.task.path == 0) {
              e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, stream_);
            } else {
              CopyBatch b;
              b.nseg = 1;
              b.pad = 0;
              b.seg[0] = CopySeg{src, dst, (unsigned long long)bytes};
              e = launch_copy(b, s.task.copy_ctas, stream_);
            }
          }
          if (e == cudaSuccess) e = cudaEventRecord(s.done, stream_);
          if (e != cudaSuccess) {
            release(best, PROXY_CUDA);
            release(i, PROXY_CUDA);
            busy_ns_ += now_ns() - w0;
            break;
          }
          s.partner = best;
          s.state = RUNNING;
          s.t0 = now;
          o.state = RUNNING;  // passive: finished by slot i
          o.partner = -2;
          busy_ns_ += now_ns() - w0;
          break;
        }
        case PARKED:
          if (now - s.t0 > limit) {  // nobody posted the other side: let the stream go and report it
            parked_--;
            release(i, PROXY_TIMEOUT);
          }
          break;
        case RUNNING: {
          if (s.partner == -2) break;  // passive half of a matched pair
          cudaError_t q = cudaEventQuery(s.done);
          if (q == cudaErrorNotReady) {
            if (now - s.t0 > limit) {
              int zero = 0;
              error_.compare_exchange_strong(zero, PROXY_TIMEOUT);  // reported; the work may still be making progress
            }
            if (now - s.t0 <= 4 * limit) break;
            // Four watchdog periods without completion: the work is considered stuck.  The stream is let go so that
            // nothing waits on this library forever; the result is undefined and the sticky error says so.
            q = cudaErrorTimeout;
          }
          const long long w0 = now_ns();
          PTRACE("pair %d: work complete (%s)", i, cudaGetErrorString(q));
          const int err = (q == cudaSuccess) ? PROXY_OK : PROXY_CUDA;
          const int partner = s.partner;
          release(i, err);
          if (partner >= 0) release(partner, err);
          busy_ns_ += now_ns() - w0;
          break;
        }
      }
    }
  }
}

}  // namespace hoccl
