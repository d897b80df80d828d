// hoccl_allreduce_static: the ring all-reduce for callers that are not allowed to allocate.
//
// Some users of this library run where device allocation is off limits: a communication thread that
// works beside training kernels and must never trigger the device-wide synchronisation an allocation
// can imply, or a process whose device memory is handed out once by a static memory planner so that no
// byte is left to ask for.  They cannot attach scratch to a communicator either, because they have none
// to give.  For them the ring's inbox and partial slots live in the fixed array below, which is part of
// the library image: every GPU that loads the library holds it from module load until the process ends.
//
// Nothing here calls cudaMalloc, cudaFree, or creates streams, events or graphs: the whole schedule is
// issued as kernel launches on the caller's stream in the planner's (topological) order.
#include <cuda_runtime.h>

#include <algorithm>
#include <mutex>

#include "../../include/hoccl.h"
#include "kernels.cuh"
#include "plan.h"

using namespace hoccl;

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table, not a
// device address: its address on a given device comes from cudaGetSymbolAddress (see scratch_base).
static __device__ __align__(256) unsigned char g_static_scratch[HOCCL_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr int kStaticSumCtas = 8;    // same SM budget for sums as the communicator's default
constexpr int kStaticCopyCtas = 32;
std::mutex g_mu;
void* g_base[kMaxDevices] = {};

// Device address of the array on the CURRENT device; looked up once per device.
cudaError_t scratch_base(int device, void** out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_base[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_base[device] = p;
  }
  *out = g_base[device];
  return cudaSuccess;
}

bool overlap(const char* a, size_t an, const char* b, size_t bn) { return an && bn && a < b + bn && b < a + an; }

}  // namespace

extern "C" hoccl_result_t hoccl_allreduce_static(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                                                 hoccl_op_t op, int R, hoccl_stream_t stream) {
  if (!send || !recv || R < 1 || R > 64) return HOCCL_ERR_INVALID_ARG;
  if (op != HOCCL_SUM) return HOCCL_ERR_UNSUPPORTED;
  const size_t e = dtype_size((int)dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  const size_t bytes = count * e;
  int n_in = 0;
  for (int r = 0; r < R; r++) {
    if (!send[r] || !recv[r]) return HOCCL_ERR_INVALID_ARG;
    if (((uintptr_t)send[r] % e) || ((uintptr_t)recv[r] % e)) return HOCCL_ERR_INVALID_ARG;
    if (send[r] == recv[r]) n_in++;
    else if (overlap((const char*)send[r], bytes, (const char*)recv[r], bytes)) return HOCCL_ERR_INVALID_ARG;
  }
  if (n_in != 0 && n_in != R) return HOCCL_ERR_INVALID_ARG;
  for (int a = 0; a < R; a++)
    for (int b = a + 1; b < R; b++) {
      const char *sa = (const char*)send[a], *sb = (const char*)send[b], *da = (const char*)recv[a], *db = (const char*)recv[b];
      if (overlap(sa, bytes, sb, bytes) || overlap(da, bytes, db, bytes) || overlap(sa, bytes, db, bytes) || overlap(da, bytes, sb, bytes))
        return HOCCL_ERR_INVALID_ARG;
    }
  if (count == 0) return HOCCL_OK;

  // one piece per ring chunk: the schedule runs on one stream, so pieces would buy nothing
  Plan P;
  unsigned char align[64];
  for (int r = 0; r < R; r++) align[r] = (unsigned char)((uintptr_t)send[r] & 15);
  if (!build_plan(&P, PLAN_ALLREDUCE, R, count, (int)dtype, n_in == R, (size_t)1 << 40, 1, align)) return HOCCL_ERR_INVALID_ARG;
  const size_t need = 2 * (size_t)R * P.slot_bytes;
  if (need > (size_t)HOCCL_STATIC_SCRATCH_BYTES) return HOCCL_ERR_SCRATCH;   // beyond the fixed maximum

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return HOCCL_ERR_CUDA;
  void* base = nullptr;
  if (P.slot_bytes && scratch_base(device, &base) != cudaSuccess) return HOCCL_ERR_CUDA;
  char* inbox0 = (char*)base;
  char* partial0 = inbox0 + (size_t)R * P.slot_bytes;
  auto addr = [&](int buf, int rank, uint64_t off) -> char* {
    switch (buf) {
      case BUF_SEND: return (char*)send[rank] + off;
      case BUF_RECV: return (char*)recv[rank] + off;
      case BUF_INBOX: return inbox0 + (size_t)rank * P.slot_bytes + off;
      default: return partial0 + (size_t)rank * P.slot_bytes + off;
    }
  };
  cudaStream_t st = (cudaStream_t)stream;
  // Groups are stored in a topological order of the plan's DAG; on a single stream that order is a valid schedule.
  for (const PlanGroup& g : P.groups) {
    for (int first = 0; first < g.num_ops; first += kMaxSegs) {
      const int n = std::min(kMaxSegs, g.num_ops - first);
      cudaError_t err;
      if (g.kind == OP_SUM) {
        SumBatch b;
        b.nseg = n;
        b.dtype = (int)dtype;
        for (int i = 0; i < n; i++) {
          const PlanOp& o = P.ops[g.first_op + first + i];
          b.seg[i] = SumSeg{addr(o.src_buf, o.rank, o.src_off), addr(o.local_buf, o.rank, o.local_off), addr(o.dst_buf, o.rank, o.dst_off),
                            (unsigned long long)(o.bytes / e)};
        }
        err = launch_sum(b, kStaticSumCtas, st);
      } else {
        CopyBatch b;
        b.nseg = n;
        b.pad = 0;
        for (int i = 0; i < n; i++) {
          const PlanOp& o = P.ops[g.first_op + first + i];
          b.seg[i] = CopySeg{addr(o.src_buf, o.rank, o.src_off), addr(o.dst_buf, o.dst_rank, o.dst_off), (unsigned long long)o.bytes};
        }
        err = launch_copy(b, kStaticCopyCtas, st);
      }
      if (err != cudaSuccess) return HOCCL_ERR_CUDA;
    }
  }
  return HOCCL_OK;
}
