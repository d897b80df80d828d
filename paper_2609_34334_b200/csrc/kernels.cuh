// Device kernels of libhoccl: the per-step chunk SUM, the SM copy used by the comparison path,
// and the bounded occupancy kernel of the "does a move need an SM" probe.  sm_100a only.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace hoccl {

constexpr int kMaxSegs = 32;       // segments (one per rank) a single batched launch can carry
constexpr int kThreads = 1024;     // threads per CTA of the copy and occupancy kernels (the sum picks 512 or 1024)

// Flattened view of a batch of segments: every segment is an element-wise head, a body of 16-byte vectors cut into
// CTA tiles, and an element-wise tail; prefix sums put the tiles (and the element-wise items) of all segments into one
// index space, so that any grid stays balanced.  The host fills it when it fills a batch (it knows every pointer and
// length), so the kernels start without a set-up phase.
struct Flat {
  unsigned long long tpre[kMaxSegs + 1];  // prefix sums of vector tiles
  unsigned long long spre[kMaxSegs + 1];  // prefix sums of element-wise items
  unsigned long long nvec[kMaxSegs];      // 16-byte vectors in the body
  unsigned int head[kMaxSegs];            // element-wise items before the body
};

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
  Flat flat;  // filled by prepare_sum_batch (the launch helpers do it themselves)
  unsigned int* smid_out = nullptr;  // diagnostics: if set, CTA b stores the id of the SM it runs on to smid_out[b]
};

// One chain segment (direct reduce-scatter): out[i] = (((s_0[i] + s_1[i]) + ...) + s_{nsrc-1}[i]) + local[i], every add one
// binary32 add rounded into the I/O dtype: the ring's order and rounding for one chunk, done by its owner in one pass.
// s_j = first + j * stride bytes: the owner's inbox slots, filled by the R-1 direct moves.
struct ChainSeg {
  const void* first;
  const void* local;
  void* out;
  unsigned long long n;       // elements
  unsigned long long stride;  // bytes, a multiple of 16
  int nsrc;                   // 1..kMaxChainSrcs
  int pad;
};
constexpr int kMaxChainSrcs = 63;
struct ChainBatch {
  int nseg;
  int dtype;
  ChainSeg seg[kMaxSegs];
  Flat flat;  // filled by prepare_chain_batch (launch_chain does it itself)
  unsigned int* smid_out = nullptr;
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
  Flat flat;  // filled by prepare_copy_batch (the launch helpers do it themselves)
  unsigned int* smid_out = nullptr;  // diagnostics, as in SumBatch
};

// One fan-out segment: every dst[first_dst + d][0..bytes), d < ndst, <- src[0..bytes).  The source is read once and stored ndst
// times (the direct all-gather on the SM path: a rank's chunk goes to all its peers, 1 + ndst instead of 2 ndst bytes of
// traffic per chunk byte).  All addresses of a segment share their 16-byte phase or the segment runs element-wise.
constexpr int kMaxFanDsts = 256;
struct FanSeg {
  const void* src;
  unsigned long long bytes;
  int first_dst, ndst;
};
struct FanBatch {
  int nseg;
  int ndst_total;
  FanSeg seg[kMaxSegs];
  void* dst[kMaxFanDsts];
  Flat flat;  // filled by prepare_fan_batch (launch_fan does it itself)
  unsigned int* smid_out = nullptr;  // diagnostics, as in SumBatch
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

// Whole-collective kernel of the SM path ("fused" setting): one cooperative launch walks the plan's groups in order,
// a grid-wide barrier between dependent groups.  This is how an SM-driven library runs a collective (one persistent
// kernel, the paper's "NCCL under an SM budget" baseline of Sec. 5), while the schedule stays rank local: MOVE into
// the receiver's inbox, then SUM out of it.  It removes the per-step launch cost that dominates small messages.
struct RingSeg {
  const void* src;     // MOVE: source; SUM: inbox
  const void* local;   // SUM: local contribution; MOVE: nullptr
  void* dst;
  unsigned long long bytes;
  // filled by the host (prepare_ring_phase): the segment's split and the running totals of its phase
  unsigned long long nvec;         // 16-byte vectors in the body
  unsigned long long tiles_end;    // tiles of this phase up to and including this segment
  unsigned long long scalars_end;  // element-wise items of this phase up to and including this segment
  unsigned int head;               // element-wise items before the body
  unsigned int pad;
};
struct RingPhase {
  int first_seg, nseg;
  int kind;            // 0 MOVE, 1 SUM
  int barrier_before;  // 1: a grid barrier separates this phase from the ones before it
};
constexpr int kRingSmallPhases = 32, kRingSmallSegs = 256;   // 16.9 KB of kernel parameters
constexpr int kRingLargePhases = 96, kRingLargeSegs = 480;   // 32.3 KB (the limit is 32,764 bytes)
constexpr unsigned kRingSpinLimit = 1u << 21;                // polls of one barrier wait before the kernel gives up (~1-2 s)
template <int NPH, int NSEG>
struct RingArgsT {
  int nphase;
  int dtype;
  int missing_arrivals;  // 0 in normal use; the self-test sets 1: every barrier then waits for a CTA that does not exist
  int pad;
  unsigned* bar;   // device words {arrivals, exits, gave-up flag}; zero between launches (the kernel resets them on exit)
  int* host_err;   // mapped pinned host word: set to 1 if a barrier wait ran out
  RingPhase phase[NPH];
  RingSeg seg[NSEG];
};
using RingArgsSmall = RingArgsT<kRingSmallPhases, kRingSmallSegs>;
using RingArgsLarge = RingArgsT<kRingLargePhases, kRingLargeSegs>;
// Largest cooperative grid of the ring kernel on the current device for the given thread count (512 or 1024).
cudaError_t ring_max_grid(int threads, int dtype, bool large, int num_sms, int* grid);
cudaError_t launch_ring(const RingArgsSmall& a, int grid, int threads, cudaStream_t stream);
cudaError_t launch_ring(const RingArgsLarge& a, int grid, int threads, cudaStream_t stream);
cudaError_t preload_ring_kernels();
// Fills nvec / head / tiles_end / scalars_end of the nseg segments of one phase for the kernel shape `threads` selects.
void prepare_ring_phase(RingSeg* seg, int nseg, int kind, int dtype, int threads);

// Enqueue helpers (return the CUDA error of the launch).
cudaError_t launch_sum(const SumBatch& batch, int ctas, cudaStream_t stream);
cudaError_t launch_copy(const CopyBatch& batch, int ctas, cudaStream_t stream);
cudaError_t launch_chain(const ChainBatch& batch, int ctas, cudaStream_t stream);
void prepare_chain_batch(ChainBatch* batch, int ctas);
// kernel and thread count that serve `batch` with `ctas` CTAs (the batch must have been prepared for the same `ctas`)
const void* chain_kernel_entry(const ChainBatch& batch, int ctas, int* threads);
// counts: two device words, zeroed by the caller; see bf16_add_selftest_kernel
cudaError_t launch_bf16_add_selftest(unsigned long long* counts, cudaStream_t stream);
cudaError_t launch_fan(const FanBatch& batch, int ctas, cudaStream_t stream);
void prepare_fan_batch(FanBatch* batch, int ctas);
const void* fan_kernel_entry(int ctas, int* threads);
// Fill batch->flat for the kernel variant that `ctas` CTAs select (needed before a batch is handed to a graph kernel node).
void prepare_sum_batch(SumBatch* batch, int ctas);
void prepare_copy_batch(CopyBatch* batch, int ctas);
// Kernel entry addresses and parameter blocks for CUDA graph kernel nodes.
const void* sum_kernel_entry(int dtype, int ctas, int* threads);
const void* copy_kernel_entry(int ctas, int* threads);
const void* graph_root_kernel_entry();   // an empty kernel (1 CTA of 32 threads): common predecessor of many root copy nodes

// Memory-port probe: `ctas` CTAs only read (mode 0) or only write (mode 1) `bytes` bytes (a multiple of 128 KiB is walked).
cudaError_t launch_port_probe(int mode, void* buf, unsigned long long bytes, int ctas, unsigned int* sink, cudaStream_t stream);

// Loads every kernel of the library on the current device (no launch).
cudaError_t preload_kernels();

// Fills every thread slot of every SM for `ns` nanoseconds (measured with %globaltimer per CTA).
// It never waits on memory or on another agent, so it always ends by itself.
cudaError_t launch_occupy_all_sms(unsigned long long ns, int num_sms, cudaStream_t stream, int* ctas_out);

}  // namespace hoccl
