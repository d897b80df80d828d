// Ring planner (see plan.h).  Ring reduce-scatter followed by ring all-gather; the paper has no
// reduction (Sec. 4 "Limitations"), so the reduce-scatter is the textbook ring with rank r ending
// as the owner of chunk r.
#include "plan.h"

#include <algorithm>

namespace hoccl {

size_t dtype_size(int dtype) { return dtype == 0 ? 4 : (dtype == 1 ? 2 : 0); }

static size_t round_up(size_t v, size_t m) { return (v + m - 1) / m * m; }

size_t slot_bytes_for(int R, size_t count, size_t elem) {
  if (R <= 1 || count == 0) return 0;
  size_t q = (count + (size_t)R - 1) / (size_t)R;
  // one chunk plus 16 bytes of alignment slack per piece; pieces are at least 1024 bytes
  return round_up(q * elem + (q * elem / 1024 + 2) * 16, 256);
}

void Plan::chunk_range(int c, size_t* lo, size_t* hi) const {
  if (kind == PLAN_ALLREDUCE) {
    size_t a = (size_t)c * chunk_elems, b = ((size_t)c + 1) * chunk_elems;
    *lo = std::min(a, count);
    *hi = std::min(b, count);
  } else {
    *lo = (size_t)c * count;
    *hi = *lo + count;
  }
}

namespace {

int mod(int a, int R) { return ((a % R) + R) % R; }

struct Builder {
  Plan* P;
  int cur_group = -1;

  int begin_group(int kind, int phase, int step, int piece) {
    PlanGroup g;
    g.kind = kind;
    g.phase = phase;
    g.step = step;
    g.piece = piece;
    g.first_op = (int)P->ops.size();
    g.num_ops = 0;
    g.chain_dep = -1;
    P->groups.push_back(g);
    cur_group = (int)P->groups.size() - 1;
    return cur_group;
  }
  // drops the group again if nothing was added to it; returns its id or -1
  int end_group() {
    int g = cur_group;
    cur_group = -1;
    if (P->groups[g].num_ops == 0) {
      P->groups.pop_back();
      return -1;
    }
    return g;
  }
  void add(PlanOp op) {
    if (op.bytes == 0) return;
    op.group = cur_group;
    P->ops.push_back(op);
    P->groups[cur_group].num_ops++;
  }
};

// piece p of a chunk of len_bytes bytes: [off, off+len)
void piece_span(const Plan& P, size_t len_bytes, int p, size_t* off, size_t* len) {
  size_t a = (size_t)P.piece_off[(size_t)p];
  size_t b = (size_t)P.piece_off[(size_t)p + 1];
  a = std::min(a, len_bytes);
  b = std::min(b, len_bytes);
  *off = a;
  *len = b - a;
}

}  // namespace

bool build_plan(Plan* plan, int kind, int R, size_t count, int dtype, bool in_place, size_t piece_bytes, int max_pieces,
                const unsigned char* send_align) {
  size_t e = dtype_size(dtype);
  if (!plan || R < 1 || e == 0 || kind < 0) return false;
  int flags = 0;
  if (kind >= 16) {
    flags = kind & ~15;
    kind &= 15;
    if (kind > PLAN_ALLTOALL || (flags & ~(PLAN_FLAG_FORWARD | PLAN_FLAG_AG_DIRECT | PLAN_FLAG_RS_DIRECT | PLAN_FLAG_GRADED))) return false;
  } else {
    if (kind > PLAN_ALLREDUCE_FWD_AGD) return false;
    if (kind == PLAN_ALLREDUCE_FWD || kind == PLAN_REDUCE_SCATTER_FWD || kind == PLAN_ALLREDUCE_FWD_AGD) flags |= PLAN_FLAG_FORWARD;
    if (kind == PLAN_ALLREDUCE_AGD || kind == PLAN_ALLGATHER_DIRECT || kind == PLAN_ALLREDUCE_FWD_AGD) flags |= PLAN_FLAG_AG_DIRECT;
    if (kind == PLAN_ALLREDUCE_FWD || kind == PLAN_ALLREDUCE_AGD || kind == PLAN_ALLREDUCE_FWD_AGD) kind = PLAN_ALLREDUCE;
    if (kind == PLAN_REDUCE_SCATTER_FWD) kind = PLAN_REDUCE_SCATTER;
    if (kind == PLAN_ALLGATHER_DIRECT) kind = PLAN_ALLGATHER;
  }
  const bool reduces = (kind == PLAN_ALLREDUCE || kind == PLAN_REDUCE_SCATTER);
  const bool gathers = (kind == PLAN_ALLREDUCE || kind == PLAN_ALLGATHER);
  const bool rs_direct = reduces && (flags & PLAN_FLAG_RS_DIRECT) && R > 1;
  const bool forward = reduces && (flags & PLAN_FLAG_FORWARD) && !rs_direct;   // the direct form has no per-step sums to forward
  const bool ag_direct = gathers && (flags & PLAN_FLAG_AG_DIRECT);
  const bool graded = reduces && (flags & PLAN_FLAG_GRADED);
  if (kind == PLAN_ALLTOALL && in_place) return false;  // an in-place exchange would need a staging copy of every block
  if (max_pieces < 1) max_pieces = 1;
  if (piece_bytes < 1024) piece_bytes = 1024;
  Plan& P = *plan;
  P = Plan();
  P.kind = kind;
  P.forward = forward;
  P.ag_direct = ag_direct;
  P.rs_direct = rs_direct;
  P.inbox_slots = rs_direct ? R - 1 : 1;
  P.uses_partial = !rs_direct;
  P.R = R;
  P.dtype = dtype;
  P.count = count;
  P.in_place = in_place;
  P.elem = e;
  P.chunk_elems = (kind == PLAN_ALLREDUCE) ? (count + (size_t)R - 1) / (size_t)R : count;
  size_t chunk_bytes = P.chunk_elems * e;
  // piece geometry: at most max_pieces pieces of equal size (multiple of 1024 bytes).  Pieces exist to overlap a
  // piece's move with another piece's sum; a pure all-gather has no sums, and on one device many small copies only
  // add per-copy cost, so it is cut no finer than 64 MiB.
  if (kind == PLAN_ALLGATHER || kind == PLAN_ALLTOALL) piece_bytes = std::max<size_t>(piece_bytes, (size_t)64 << 20);
  size_t want = (chunk_bytes + piece_bytes - 1) / piece_bytes;
  size_t np = std::max<size_t>(1, std::min<size_t>(want, (size_t)max_pieces));
  size_t plen = round_up((chunk_bytes + np - 1) / np, 1024);
  // pieces of 256 KiB or more are whole multiples of 128 KiB (the copy kernels' tile): measured on B200, R = 8, 40 MiB per rank,
  // pieces of 1708 or 854 KiB (a third, a sixth of the ring chunk) ran 15 % slower than the same schedule with 1280 or 640 KiB
  if (np > 1 && plen >= ((size_t)256 << 10)) plen = round_up(plen, (size_t)128 << 10);
  if (plen == 0) plen = 1024;
  P.piece_bytes = plen;
  P.pieces = (int)std::max<size_t>(1, (chunk_bytes + plen - 1) / plen);
  P.piece_off.assign((size_t)P.pieces + 1, 0);
  for (int p = 0; p <= P.pieces; p++) P.piece_off[(size_t)p] = std::min<uint64_t>((uint64_t)p * plen, chunk_bytes);
  if (graded && P.pieces >= 3 && plen >= ((size_t)256 << 10)) {
    // Graded pieces, in units of 128 KiB: weights 1/3, 2/3, 1, ..., 1, 2/3, 1/3 (with three or four pieces only the outer ones
    // shrink).  The count stays; the middle pieces grow by what the outer ones give up.
    const size_t u = (size_t)128 << 10;
    const size_t units = (chunk_bytes + u - 1) / u;
    const int n = P.pieces;
    std::vector<double> w((size_t)n, 1.0);
    const int ramp = n >= 6 ? 2 : 1;
    for (int k = 0; k < ramp; k++) {
      w[(size_t)k] = w[(size_t)(n - 1 - k)] = (double)(k + 1) / (double)(ramp + 1);
    }
    double wsum = 0;
    for (double x : w) wsum += x;
    std::vector<size_t> sz((size_t)n, 0);
    size_t used = 0;
    for (int k = 0; k < n; k++) {
      sz[(size_t)k] = std::max<size_t>(1, (size_t)((double)units * w[(size_t)k] / wsum));
      used += sz[(size_t)k];
    }
    // what rounding left over goes to (or comes from) the middle pieces, one unit at a time
    for (int k = ramp; used < units; k = (k + 1 - ramp) % std::max(1, n - 2 * ramp) + ramp) {
      sz[(size_t)k]++;
      used++;
    }
    size_t guard = 0;
    for (int k = ramp; used > units && guard < units * (size_t)n; k = (k + 1 - ramp) % std::max(1, n - 2 * ramp) + ramp, guard++) {
      if (sz[(size_t)k] > 1) {
        sz[(size_t)k]--;
        used--;
      }
    }
    size_t off = 0, biggest = 0;
    for (int k = 0; k < n; k++) {
      P.piece_off[(size_t)k] = std::min<uint64_t>(off, chunk_bytes);
      off += sz[(size_t)k] * u;
      biggest = std::max(biggest, sz[(size_t)k] * u);
    }
    P.piece_off[(size_t)n] = chunk_bytes;
    P.piece_bytes = biggest;
  }
  // Slack between the regions of consecutive pieces inside a scratch slot: 16 bytes hold the phase shift (below); pieces of
  // 16 KiB or more get 128, so that every region starts on a 128-byte line like the operands it is summed with.  (With 16 the
  // region of piece p sat 16 p bytes off the line grid: a warp's 512-byte load then touched five lines instead of four, and the
  // chain sum of every piece but the first ran ~20 % slower.)  Both stay inside slot_bytes_for: 128 per 16 KiB is 1/128 of the
  // chunk, the bound grants 1/64.
  const size_t slack = (P.pieces > 1 && P.piece_bytes >= ((size_t)16 << 10)) ? 128 : 16;
  P.slot_bytes = (kind == PLAN_ALLGATHER || kind == PLAN_ALLTOALL || R == 1) ? 0 : round_up(chunk_bytes + slack * (size_t)P.pieces, 256);
  if (count == 0) return true;
  // Where piece p of chunk c sits inside a scratch slot of rank r: every piece has its own region with `slack`
  // bytes of slack, and inside it the data is shifted by the 16-byte phase of the operand it is summed with
  // (rank r's send data of chunk c), so that the three SUM operands stay congruent modulo 16.
  auto slot_off = [&](int r, int c, int p) -> uint64_t {
    size_t lo, hi;
    P.chunk_range(c, &lo, &hi);
    size_t phase = ((send_align ? (size_t)(send_align[r] & 15) : 0) + lo * e) & 15;
    return P.piece_off[(size_t)p] + (uint64_t)p * slack + phase;
  };

  Builder B{&P};
  const int np_i = P.pieces;

  if (R == 1) {
    if (!in_place) {
      for (int p = 0; p < np_i; p++) {
        size_t off, len;
        piece_span(P, chunk_bytes, p, &off, &len);
        B.begin_group(OP_MOVE, PHASE_OWN, 0, p);
        B.add(PlanOp{OP_MOVE, PHASE_OWN, 0, p, 0, 0, 0, BUF_SEND, BUF_RECV, -1, off, off, 0, len, 0});
        B.end_group();
      }
    }
    return true;
  }

  if (kind == PLAN_ALLTOALL) {
    // All-to-all as R-1 permutation stages (the matching-peeling view of the paper's stage decomposition, Sec. 3.4:
    // stage k is the contention-free matching r -> r+k of the uniform traffic matrix) plus the own block.  All flows
    // have the same size, so chunk service is plain round-robin over ranks.  No dependencies: blocks are disjoint.
    for (int p = 0; p < np_i; p++) {
      B.begin_group(OP_MOVE, PHASE_OWN, 0, p);
      for (int r = 0; r < R; r++) {
        size_t off, len;
        piece_span(P, chunk_bytes, p, &off, &len);
        uint64_t blk = (uint64_t)r * count * e + off;
        B.add(PlanOp{OP_MOVE, PHASE_OWN, 0, p, r, r, r, BUF_SEND, BUF_RECV, -1, blk, blk, 0, len, 0});
      }
      B.end_group();
    }
    for (int k = 1; k < R; k++)
      for (int p = 0; p < np_i; p++) {
        B.begin_group(OP_MOVE, PHASE_A2A, k, p);
        for (int r = 0; r < R; r++) {
          int d = (r + k) % R;
          size_t off, len;
          piece_span(P, chunk_bytes, p, &off, &len);
          B.add(PlanOp{OP_MOVE, PHASE_A2A, k, p, r, d, d, BUF_SEND, BUF_RECV, -1, (uint64_t)d * count * e + off,
                       (uint64_t)r * count * e + off, 0, len, 0});
        }
        B.end_group();
      }
    return true;
  }

  std::vector<int> last_sum(np_i, -1);   // SUM group of the previous step, per piece
  std::vector<int> final_sum(np_i, -1);  // SUM group of step R-2, per piece
  int prev_sum_group = -1;

  if (rs_direct) {
    // ---- direct MOVE(k, r, p): rank r sends its contribution to chunk d = r + k to rank d, k = 1..R-1 (stage k is the
    // contention-free permutation r -> r+k).  Rank d keeps source (d+1+j) in inbox slot j, the order in which the ring
    // would have added them.  All moves of a piece form one group: none waits for anything.
    // ---- CHAIN(d, p): out = (((s_0 + s_1) + ...) + s_{R-2}) + own contribution, one pass, rounded after every add.
    for (int p = 0; p < np_i; p++) {
      int gm = B.begin_group(OP_MOVE, PHASE_RS, 0, p);
      for (int k = 1; k < R; k++)
        for (int r = 0; r < R; r++) {
          int d = (r + k) % R;
          size_t lo, hi, off, len;
          P.chunk_range(d, &lo, &hi);
          piece_span(P, (hi - lo) * e, p, &off, &len);
          PlanOp op{OP_MOVE, PHASE_RS, k - 1, p, r, d, d, BUF_SEND, BUF_INBOX, -1, lo * e + off,
                    (uint64_t)(R - 1 - k) * P.slot_bytes + slot_off(d, d, p), 0, len, 0};
          B.add(op);
        }
      gm = B.end_group();
      int gs = B.begin_group(OP_CHAIN, PHASE_RS, R - 2, p);
      for (int d = 0; d < R; d++) {
        size_t lo, hi, off, len;
        P.chunk_range(d, &lo, &hi);
        piece_span(P, (hi - lo) * e, p, &off, &len);
        PlanOp op{OP_CHAIN, PHASE_RS, R - 2, p, d, d, d, BUF_INBOX, BUF_RECV, BUF_SEND, slot_off(d, d, p),
                  (kind == PLAN_ALLREDUCE ? lo * e : 0) + off, lo * e + off, len, 0};
        op.nsrc = R - 1;
        op.src_stride = P.slot_bytes;
        B.add(op);
      }
      gs = B.end_group();
      if (gs >= 0) {
        if (gm >= 0) P.groups[gs].deps.push_back(gm);
        P.groups[gs].chain_dep = prev_sum_group;
        prev_sum_group = gs;
        final_sum[p] = gs;
      }
    }
  } else if (kind != PLAN_ALLGATHER) {
    for (int s = 0; s <= R - 2; s++) {
      for (int p = 0; p < np_i; p++) {
        // ---- MOVE(s, r, p): chunk c = (r-1-s) mod R leaves rank r for the inbox of rank r+1.
        // Forward variant: only step 0 moves; afterwards SUM(s-1) has already written into the next rank's slot.  The
        // two scratch slots of a rank then alternate as inbox (even steps: INBOX, odd steps: PARTIAL), because a SUM
        // launch reads every rank's current inbox while it writes every rank's next one.
        int gm = B.begin_group(OP_MOVE, PHASE_RS, s, p);
        for (int r = 0; r < R && !(forward && s > 0); r++) {
          int c = mod(r - 1 - s, R);
          size_t lo, hi, off, len;
          P.chunk_range(c, &lo, &hi);
          piece_span(P, (hi - lo) * e, p, &off, &len);
          PlanOp op{OP_MOVE, PHASE_RS, s, p, r, (r + 1) % R, c, s == 0 ? BUF_SEND : BUF_PARTIAL, BUF_INBOX, -1,
                    s == 0 ? lo * e + off : slot_off(r, c, p), slot_off((r + 1) % R, c, p), 0, len, 0};
          B.add(op);
        }
        gm = B.end_group();
        if (gm >= 0 && s > 0 && last_sum[p] >= 0) P.groups[gm].deps.push_back(last_sum[p]);
        // ---- SUM(s, r, p): chunk c = (r-2-s) mod R: inbox + own contribution
        int gs = B.begin_group(OP_SUM, PHASE_RS, s, p);
        for (int r = 0; r < R; r++) {
          int c = mod(r - 2 - s, R);
          size_t lo, hi, off, len;
          P.chunk_range(c, &lo, &hi);
          piece_span(P, (hi - lo) * e, p, &off, &len);
          bool last = (s == R - 2);
          uint64_t out_off = last ? ((kind == PLAN_ALLREDUCE ? lo * e : 0) + off) : slot_off(r, c, p);
          PlanOp op{OP_SUM, PHASE_RS, s, p, r, r, c, BUF_INBOX, last ? BUF_RECV : BUF_PARTIAL, BUF_SEND,
                    slot_off(r, c, p), out_off, lo * e + off, len, 0};
          if (forward) {
            op.src_buf = (s % 2 == 0) ? BUF_INBOX : BUF_PARTIAL;
            if (!last) {
              op.dst_rank = (r + 1) % R;
              op.dst_buf = ((s + 1) % 2 == 0) ? BUF_INBOX : BUF_PARTIAL;
              op.dst_off = slot_off((r + 1) % R, c, p);
            }
          }
          B.add(op);
        }
        gs = B.end_group();
        if (gs >= 0) {
          if (gm >= 0) P.groups[gs].deps.push_back(gm);
          if (forward && s > 0 && last_sum[p] >= 0) P.groups[gs].deps.push_back(last_sum[p]);
          P.groups[gs].chain_dep = prev_sum_group;
          prev_sum_group = gs;
          last_sum[p] = gs;
          if (s == R - 2) final_sum[p] = gs;
        }
      }
    }
  }

  if (kind != PLAN_REDUCE_SCATTER) {
    const bool standalone = (kind == PLAN_ALLGATHER);
    if (standalone && !in_place) {
      // own chunk: Y_r[chunk r] <- X_r (independent of the ring: step 0 reads X_r directly)
      for (int p = 0; p < np_i; p++) {
        B.begin_group(OP_MOVE, PHASE_OWN, 0, p);
        for (int r = 0; r < R; r++) {
          size_t lo, hi, off, len;
          P.chunk_range(r, &lo, &hi);
          piece_span(P, (hi - lo) * e, p, &off, &len);
          B.add(PlanOp{OP_MOVE, PHASE_OWN, 0, p, r, r, r, BUF_SEND, BUF_RECV, -1, off, lo * e + off, 0, len, 0});
        }
        B.end_group();
      }
    }
    if (ag_direct) {
      // ---- direct AG MOVE(k, r, p): rank r sends its own final chunk r to rank r+k, k = 1..R-1.  Stage k is the
      // contention-free permutation r -> r+k; the stages do not depend on each other, only on the chunk being final.
      for (int p = 0; p < np_i; p++)
        for (int k = 1; k < R; k++) {
          int g = B.begin_group(OP_MOVE, PHASE_AG, k - 1, p);
          for (int r = 0; r < R; r++) {
            size_t lo, hi, off, len;
            P.chunk_range(r, &lo, &hi);
            piece_span(P, (hi - lo) * e, p, &off, &len);
            bool from_send = standalone && !in_place;
            B.add(PlanOp{OP_MOVE, PHASE_AG, k - 1, p, r, (r + k) % R, r, from_send ? BUF_SEND : BUF_RECV, BUF_RECV, -1,
                         from_send ? off : lo * e + off, lo * e + off, 0, len, 0});
          }
          g = B.end_group();
          if (g >= 0 && !standalone && final_sum[p] >= 0) P.groups[g].deps.push_back(final_sum[p]);
        }
      return true;
    }
    std::vector<int> last_ag(np_i, -1);
    for (int s = 0; s <= R - 2; s++) {
      for (int p = 0; p < np_i; p++) {
        // ---- AG MOVE(s, r, p): final chunk c = (r-s) mod R goes from Y_r to the same place in Y_{r+1}
        int g = B.begin_group(OP_MOVE, PHASE_AG, s, p);
        for (int r = 0; r < R; r++) {
          int c = mod(r - s, R);
          size_t lo, hi, off, len;
          P.chunk_range(c, &lo, &hi);
          piece_span(P, (hi - lo) * e, p, &off, &len);
          bool from_send = standalone && !in_place && s == 0;
          B.add(PlanOp{OP_MOVE, PHASE_AG, s, p, r, (r + 1) % R, c, from_send ? BUF_SEND : BUF_RECV, BUF_RECV, -1,
                       from_send ? off : lo * e + off, lo * e + off, 0, len, 0});
        }
        g = B.end_group();
        if (g >= 0) {
          if (s == 0) {
            if (!standalone && final_sum[p] >= 0) P.groups[g].deps.push_back(final_sum[p]);
          } else if (last_ag[p] >= 0) {
            P.groups[g].deps.push_back(last_ag[p]);
          }
          last_ag[p] = g;
        }
      }
    }
  }
  return true;
}

}  // namespace hoccl
