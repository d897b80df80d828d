// Device kernels of libhoccl: the per-step chunk SUM, the SM copy used by the comparison path,
// and the bounded occupancy kernel of the "does a move need an SM" probe.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace hoccl {

constexpr int kMaxSegs = 32;       // segments (one per rank) a single batched launch can carry
constexpr int kThreads = 1024;     // threads per CTA of the copy and occupancy kernels (the sum picks 512 or 1024)

// One SUM segment: out[i] = rn_T(f32(inbox[i]) + f32(local[i])), i < n (elements).
struct SumSeg {
  const void* inbox;
  const void* local;
  void* out;
  unsigned long long n;
};
struct SumBatch {
  int nseg;
  int dtype;  // 0 fp32, 1 bf16
  SumSeg seg[kMaxSegs];
};

// One copy segment: dst[0..bytes) <- src[0..bytes).
struct CopySeg {
  const void* src;
  void* dst;
  unsigned long long bytes;
};
struct CopyBatch {
  int nseg;
  int pad;
  CopySeg seg[kMaxSegs];
};

// One-pass variant of the ring reduction (comparison point, not rank local): every element is reduced in registers in
// the ring's order, chunk c as ((x_{c+1} + x_{c+2}) + ... ) + x_c with a rounding to the I/O dtype after every add, and
// written to its destinations directly.  Same bits as the ring, R reads + R (or 1) writes per element instead of 7(R-1).
constexpr int kMaxOnePassRanks = 64;
struct OnePassArgs {
  int R;
  int dtype;
  int write_all;             // 1: all-reduce (every y[r] gets every chunk); 0: reduce-scatter (chunk c goes to y[c] at offset 0)
  int pad;
  unsigned long long count;  // elements of the reduced vector (all-reduce: per rank; reduce-scatter: R * per-rank count)
  unsigned long long q;      // elements of a full ring chunk
  const void* x[kMaxOnePassRanks];
  void* y[kMaxOnePassRanks];
};
cudaError_t launch_onepass(const OnePassArgs& args, int ctas, cudaStream_t stream);

// Enqueue helpers (return the CUDA error of the launch).
cudaError_t launch_sum(const SumBatch& batch, int ctas, cudaStream_t stream);
cudaError_t launch_copy(const CopyBatch& batch, int ctas, cudaStream_t stream);
// Kernel entry addresses and parameter blocks for CUDA graph kernel nodes.
const void* sum_kernel_entry(int dtype, int ctas, int* threads);
const void* copy_kernel_entry(int ctas, int* threads);

// Loads every kernel of the library on the current device (no launch).
cudaError_t preload_kernels();

// Fills every thread slot of every SM for `ns` nanoseconds (measured with %globaltimer per CTA).
// It never waits on memory or on another agent, so it always ends by itself.
cudaError_t launch_occupy_all_sms(unsigned long long ns, int num_sms, cudaStream_t stream, int* ctas_out);

}  // namespace hoccl
