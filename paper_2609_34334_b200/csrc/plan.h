// Host-side planner: a ring collective becomes a DAG of groups of chunk-piece operations.
//
// The paper's collective scheduler turns a collective into stages of point-to-point flows and cuts
// the flows into fixed-size chunks for the copy queue (Sec. 3.4, "Topo-aware flow schedule" and
// "Flow-size-aware chunk scheduling").  On one device every ring step is one permutation stage
// (rank r -> rank r+1) and all flows of a stage have the same size, so the weighted interleaving
// degenerates to round-robin over ranks.  Pieces of a chunk give the pipelining of Sec. 3.3
// ("chunk pipelining"): the move of piece p+1 overlaps the sum of piece p.
//
// Pure C++: no CUDA types, testable without a GPU.
#pragma once
#include <cstddef>
#include <cstdint>
#include <vector>

namespace hoccl {

enum PlanKind { PLAN_ALLREDUCE = 0, PLAN_REDUCE_SCATTER = 1, PLAN_ALLGATHER = 2, PLAN_ALLTOALL = 3,
                // comparison variants: the SUM of step s writes straight into the next rank's inbox (no moves after step 0)
                PLAN_ALLREDUCE_FWD = 4, PLAN_REDUCE_SCATTER_FWD = 5,
                // direct all-gather: the all-gather's traffic matrix (every rank sends its chunk to every other rank) cut into
                // the R-1 permutation stages r -> r+k (the stage decomposition of Sec. 3.4) instead of R-1 dependent ring hops
                PLAN_ALLREDUCE_AGD = 6, PLAN_ALLGATHER_DIRECT = 7, PLAN_ALLREDUCE_FWD_AGD = 8 /* both variants */ };
// General form of a variant: base kind (0..3) | flags.  The numbered variants above are shorthands for some combinations.
enum PlanFlag { PLAN_FLAG_FORWARD = 16, PLAN_FLAG_AG_DIRECT = 32,
                // direct reduce-scatter: the reduce-scatter's traffic matrix (rank r owes chunk d to rank d) cut into the R-1
                // permutation stages r -> r+k (Sec. 3.4); rank d keeps the R-1 contributions in R-1 inbox slots and sums them
                // in the ring's order in one pass (OP_CHAIN): same bits, 2 S (R-1) + S (R+1) instead of 5 S (R-1) bytes
                PLAN_FLAG_RS_DIRECT = 64,
                // graded pieces (reductions): the first and the last pieces of a chunk are smaller than the middle ones (a third,
                // two thirds of a middle piece), so that less of the pipeline's fill and drain (the moves in front of the first
                // sum and behind the last one) is exposed.  Pieces of 256 KiB or more only; same operations, same bits.
                PLAN_FLAG_GRADED = 128 };
enum OpKind { OP_MOVE = 0, OP_SUM = 1,
              // out = (((s_0 + s_1) + ...) + s_{nsrc-1}) + local, rounded to the I/O dtype after every add; s_j at src_off + j * src_stride
              OP_CHAIN = 2 };
enum BufKind { BUF_SEND = 0, BUF_RECV = 1, BUF_INBOX = 2, BUF_PARTIAL = 3 };
enum Phase { PHASE_RS = 0, PHASE_AG = 1, PHASE_OWN = 2, PHASE_A2A = 3 };

struct PlanOp {
  int kind;
  int phase, step, piece;
  int rank, dst_rank, chunk;
  int src_buf, dst_buf, local_buf;
  uint64_t src_off, dst_off, local_off;  // bytes from the start of the buffer (scratch: from the start of the rank's slot)
  uint64_t bytes;
  int group;
  int nsrc = 1;             // OP_CHAIN: number of inbox operands (R-1)
  uint64_t src_stride = 0;  // OP_CHAIN: bytes between consecutive inbox operands (one scratch slot)
};

struct PlanGroup {
  int kind;  // OpKind of every op in the group
  int phase, step, piece;
  int first_op, num_ops;
  std::vector<int> deps;  // data dependencies (group ids, all smaller than this group's id)
  int chain_dep;          // previous SUM group in issue order (-1 if none): keeps SUM launches serial
};

struct Plan {
  int kind = 0, R = 0, dtype = 0;  // kind: the base collective (forward variants are folded into it, see `forward`)
  bool forward = false;            // fused sum-and-forward variant (not rank local)
  bool ag_direct = false;          // all-gather phase as R-1 independent permutation stages (rank local: rank r sends its own chunk)
  bool rs_direct = false;          // reduce-scatter phase as R-1 independent permutation stages + one chain sum per rank
  int inbox_slots = 1;             // scratch slots of one rank's inbox (rs_direct: R-1); the partial slots follow all inboxes
  bool uses_partial = true;        // false: no partial slots in the scratch (rs_direct)
  size_t scratch_need() const { return (size_t)R * slot_bytes * ((size_t)inbox_slots + (uses_partial ? 1 : 0)); }
  size_t count = 0;
  bool in_place = false;
  size_t elem = 4;
  size_t chunk_elems = 0;   // q: elements of a full ring chunk
  size_t piece_bytes = 0;   // bytes of the largest piece (multiple of 1024 unless the chunk is one piece)
  int pieces = 1;
  std::vector<uint64_t> piece_off;   // pieces + 1 byte offsets inside a full ring chunk; piece p is [piece_off[p], piece_off[p+1])
  size_t slot_bytes = 0;    // bytes of one scratch slot (inbox or partial) of one rank, padded
  std::vector<PlanOp> ops;
  std::vector<PlanGroup> groups;

  // element range [lo, hi) of ring chunk c inside the rank buffer that holds all R chunks
  void chunk_range(int c, size_t* lo, size_t* hi) const;
};

size_t dtype_size(int dtype);  // 0 if unknown

// upper bound of the scratch slot size (bytes) for one rank and one slot kind, whatever the piece
// settings: one ring chunk + 16 bytes of alignment slack per piece, rounded up to 256
size_t slot_bytes_for(int R, size_t count_allreduce_convention, size_t elem);

// Returns false on invalid arguments.  `count` follows the collective's convention.  send_align (R entries
// or NULL for "all 16-byte aligned") gives the low 4 bits of each rank's send pointer; it only decides where
// inside its scratch region a piece is placed.
bool build_plan(Plan* plan, int kind, int R, size_t count, int dtype, bool in_place, size_t piece_bytes, int max_pieces,
                const unsigned char* send_align);

}  // namespace hoccl
