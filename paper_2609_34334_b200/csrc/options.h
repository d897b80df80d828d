// How the settings of a communicator combine for one call: which schedule (plan kind and flags), which executor, and on
// which move route it runs.  One function decides this for every entry point, so that a combination is either served as
// asked or refused (HOCCL_ERR_UNSUPPORTED); nothing is dropped silently.  Pure host code: testable without a GPU.
//
// Rules (value 1 = asked for, 2 = automatic, which yields to anything asked for):
//   handshake   needs HOCCL_PATH_SM (a driver copy issued by the proxy can queue up behind the parked stream's own copies);
//               it replays graphs through the proxy, so "onepass" and "fused" cannot be combined with it.
//   onepass     applies to all-reduce and reduce-scatter calls only and replaces the whole schedule there: "forward",
//               "fused", "rs_direct" = 1 and "ag_direct" = 1 cannot be combined with it for those calls.  It ignores the path.
//   fused       one cooperative kernel on HOCCL_PATH_SM: refused on the other paths; it has no chain phase and does not
//               forward, so "rs_direct" = 1 is refused with it; "forward" with "fused" is served (the ring kernel walks the
//               forward plan).  It ignores "use_graph".
//   roles       all-reduce and reduce-scatter calls as ONE cooperative kernel with summing and moving CTAs (roles.cu).  It runs
//               the direct schedule on HOCCL_PATH_SM for 2 to 8 ranks: refused on the other paths, for other rank counts, with
//               "handshake", "onepass", "forward", "fused", "rs_direct" = 0 and (all-reduce) "ag_direct" = 0.  Like "rs_direct"
//               = 1 it needs the scratch of the direct form (HOCCL_ERR_SCRATCH otherwise).  Other calls ignore it; so does the
//               pipelined host entry.  It ignores "use_graph".
//   forward     applies to all-reduce and reduce-scatter; "rs_direct" = 1 is refused with it (the direct form has no steps
//               to forward between).
//   rs_direct   2 takes the direct reduce-scatter when nothing above excludes it and the attached scratch holds its R - 1
//               inbox slots per rank; 1 asks for it (the call fails with HOCCL_ERR_SCRATCH later if the scratch is too small).
//   ag_direct   2 takes the direct all-gather on HOCCL_PATH_SM and HOCCL_PATH_CE_HOST always, on HOCCL_PATH_CE while a
//               ring chunk is at most 64 MiB.
//   use_graph   chooses between graph replay and the stream executor where neither handshake nor fused decides.
//   ce_small_bytes  on HOCCL_PATH_CE a call whose per-rank message is at most this many bytes issues its moves as batched
//               launches of the copy kernel with "ce_small_ctas" CTAs (the route of HOCCL_PATH_SM): on one device a driver
//               copy spares no SM and costs microseconds to start.  0 switches this off.
#pragma once
#include <cstddef>

#include "../../include/hoccl.h"

namespace hoccl {

enum Executor { EXEC_GRAPH = 0, EXEC_STREAMS = 1, EXEC_ONE_KERNEL = 2, EXEC_ONEPASS = 3, EXEC_PROXY = 4, EXEC_ROLES = 5 };

struct OptionsIn {
  int kind;          // PlanKind base: 0 all-reduce, 1 reduce-scatter, 2 all-gather, 3 all-to-all
  int R;
  size_t count;      // the collective's own convention
  int dtype;
  int path;          // hoccl_path_t
  long onepass, forward, fused, rs_direct, ag_direct, handshake, use_graph;
  long ce_small_bytes, ce_small_ctas, copy_ctas;
  size_t scratch_bytes;   // attached scratch (0: none)
  int host_call;          // hoccl_host_allreduce
  long roles = 0;
};

struct OptionsOut {
  int plan_kind;     // base kind | PlanFlag bits
  int executor;      // Executor
  int path;          // the move route the call runs on (HOCCL_PATH_SM for a small message on HOCCL_PATH_CE)
  long copy_ctas;    // CTAs of its copy launches
  int small_switch;  // 1 if the small-message rule changed the route
};

hoccl_result_t resolve_options(const OptionsIn& in, OptionsOut* out);

}  // namespace hoccl
