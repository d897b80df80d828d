// See options.h.
#include "options.h"

#include "plan.h"

namespace hoccl {

hoccl_result_t resolve_options(const OptionsIn& in, OptionsOut* out) {
  if (!out || in.R < 1 || in.kind < PLAN_ALLREDUCE || in.kind > PLAN_ALLTOALL) return HOCCL_ERR_INVALID_ARG;
  const size_t e = dtype_size(in.dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  const bool reduction = in.kind == PLAN_ALLREDUCE || in.kind == PLAN_REDUCE_SCATTER;
  const bool gathers = in.kind == PLAN_ALLREDUCE || in.kind == PLAN_ALLGATHER;

  // ---- the move route
  int path = in.path;
  long copy_ctas = in.copy_ctas;
  int small_switch = 0;
  if (in.handshake && in.path != HOCCL_PATH_SM) return HOCCL_ERR_UNSUPPORTED;
  const size_t per_rank = in.kind == PLAN_ALLREDUCE ? in.count * e : in.count * (size_t)in.R * e;
  if (in.path == HOCCL_PATH_CE && in.ce_small_bytes > 0 && per_rank <= (size_t)in.ce_small_bytes && !in.host_call) {
    path = HOCCL_PATH_SM;
    copy_ctas = in.ce_small_ctas;
    small_switch = 1;
  }

  // ---- what was asked for must fit together
  const bool onepass = in.onepass && reduction;
  if (in.handshake && (in.onepass || in.fused)) return HOCCL_ERR_UNSUPPORTED;
  if (in.fused && in.path != HOCCL_PATH_SM) return HOCCL_ERR_UNSUPPORTED;
  if (onepass && (in.forward || in.fused || in.rs_direct == 1 || (in.ag_direct == 1 && in.kind == PLAN_ALLREDUCE)))
    return HOCCL_ERR_UNSUPPORTED;
  if (reduction && in.rs_direct == 1 && (in.forward || in.fused)) return HOCCL_ERR_UNSUPPORTED;

  const bool roles = in.roles && reduction && !in.host_call;
  if (roles && (in.path != HOCCL_PATH_SM || in.R < 2 || in.R > 8 || in.handshake || in.onepass || in.forward || in.fused || in.rs_direct == 0 ||
                (in.kind == PLAN_ALLREDUCE && in.ag_direct == 0)))
    return HOCCL_ERR_UNSUPPORTED;

  const bool forward = in.forward && reduction;
  const bool fused = in.fused && !in.host_call;   // the pipelined host entry runs its pieces as graphs
  bool direct_rs = reduction && (in.rs_direct == 1 || roles);
  if (reduction && in.rs_direct == 2 && in.R > 1 && !forward && !in.fused && !onepass && !roles) {
    const size_t cnt = in.kind == PLAN_ALLREDUCE ? in.count : in.count * (size_t)in.R;
    direct_rs = in.scratch_bytes >= (size_t)(in.R - 1) * (size_t)in.R * slot_bytes_for(in.R, cnt, e);
  }
  bool direct_ag = gathers && (in.ag_direct == 1 || roles);
  if (gathers && in.ag_direct == 2) {
    const size_t q = in.kind == PLAN_ALLREDUCE ? (in.count + in.R - 1) / in.R : in.count;
    direct_ag = path != HOCCL_PATH_CE || q * e <= ((size_t)64 << 20);
  }

  out->plan_kind = in.kind | (forward ? PLAN_FLAG_FORWARD : 0) | (direct_ag ? PLAN_FLAG_AG_DIRECT : 0) | (direct_rs ? PLAN_FLAG_RS_DIRECT : 0);
  if (onepass) out->executor = EXEC_ONEPASS;
  else if (in.handshake) out->executor = EXEC_PROXY;
  else if (fused) out->executor = EXEC_ONE_KERNEL;
  else if (roles) out->executor = EXEC_ROLES;
  else out->executor = in.use_graph ? EXEC_GRAPH : EXEC_STREAMS;
  out->path = path;
  out->copy_ctas = copy_ctas;
  out->small_switch = small_switch;
  return HOCCL_OK;
}

}  // namespace hoccl
