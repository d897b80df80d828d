/*
 * hoccl_diag.h - diagnostics of libhoccl.so: measurements, self-tests, direct kernel launches and host-only inspection
 * of what the planner and the option rules produce.  None of this is needed to run a collective (hoccl.h is); it is
 * what the tests, the microbenchmarks and the benchmark's evidence lines call.  Same conventions as hoccl.h.
 */
#ifndef HOCCL_DIAG_H_
#define HOCCL_DIAG_H_

#include "hoccl.h"

#ifdef __cplusplus
extern "C" {
#endif

/* ---------------------------------------------------------------- measurements ----------------- */

/*
 * Measures whether a MOVE of `bytes` bytes on the given path needs an SM.  A kernel that fills every
 * thread slot of every SM sleeps for a fixed `spin_us` microseconds (bounded; it never waits on
 * anything) while the move is enqueued on another stream; *needs_sm is 1 if the move finished only
 * after that kernel ended, 0 if it finished while all SMs were taken.  *move_end_us is the move's
 * completion time measured from the kernel's start.  Synchronises the device.  This is the
 * single-GPU form of the paper's claim that copy-engine transfers occupy no SM (Sec. 2.3).
 * src and dst are device buffers of at least `bytes` bytes.  On the CE path src may also be PINNED HOST
 * memory: a host-to-device copy is driven by a copy engine, which makes it the control of the measurement
 * (it must report needs_sm = 0).
 */
hoccl_result_t hoccl_probe_move_needs_sm(hoccl_comm_t comm, hoccl_path_t path, void* dst, const void* src, size_t bytes,
                                         int spin_us, int* needs_sm, double* move_end_us);

/*
 * The same measurement for every way the CUDA API offers to move bytes inside one device, one after the other:
 * cudaMemcpyAsync, cudaMemcpyPeerAsync with both ends on this device, cuMemcpyDtoDAsync, a memcpy node of a CUDA
 * graph, cudaMemcpy2DAsync, cudaMemsetAsync, this library's copy_kernel, and as controls a 32-bit stream memory
 * write (what the paper's handshake uses, Listing 1) and, when pinned host staging is attached
 * (hoccl_comm_set_host_staging, at least `bytes` bytes), a copy in each direction between device and pinned host.
 * Writes one record per route that could be tried (at most max_out) and their number to *n_out.
 * dst and src are disjoint device buffers of `bytes` bytes (bytes >= 4; dst is overwritten).  Synchronises the device.
 * Errors: INVALID_ARG (null pointer, bytes < 4, spin_us outside [100, 20000]), CUDA.
 */
typedef struct {
  char name[56];   /* which route */
  int needs_sm;    /* 1: finished only after the SM-occupying kernel ended */
  double end_us;   /* completion time, measured from the start of that kernel */
} hoccl_route_probe_t;
hoccl_result_t hoccl_probe_copy_routes(hoccl_comm_t comm, void* dst, const void* src, size_t bytes, int spin_us,
                                       hoccl_route_probe_t* out, int max_out, int* n_out);

/*
 * Direct launches of the two kernels (used by kernel-level tests and roofline measurements).
 *  hoccl_sum_launch : out[i] = round_to_dtype(float(inbox[i]) + float(local[i])), i < count, with `ctas` CTAs.
 *  hoccl_copy_launch: dst bytes <- src bytes with `ctas` CTAs.
 *  hoccl_fanout_launch: dsts[d] bytes <- src bytes for every d < ndst with `ctas` CTAs; every source byte is read once
 *                    and stored ndst times (the move of the direct all-gather on the SM path, see "ag_direct").  `dsts`
 *                    is a HOST array of ndst (1..256) device pointers; destinations must not overlap the source or each
 *                    other.  Destinations whose address differs from the source's modulo 16 are copied byte by byte.
 * All pointers are device pointers aligned to the element size (any byte alignment for the copies).
 */
hoccl_result_t hoccl_sum_launch(const void* inbox, const void* local, void* out, size_t count, hoccl_dtype_t dtype,
                                int ctas, hoccl_stream_t stream);
hoccl_result_t hoccl_copy_launch(const void* src, void* dst, size_t bytes, int ctas, hoccl_stream_t stream);
hoccl_result_t hoccl_fanout_launch(const void* src, void* const* dsts, int ndst, size_t bytes, int ctas, hoccl_stream_t stream);
/* Direct launch of the chain sum of the direct reduce-scatter ("rs_direct"): out[i] = (((s_0[i] + s_1[i]) + ...) + s_{nsrc-1}[i])
 * + local[i], i < count, every add rounded into `dtype`; s_j = first + j * stride_bytes (a multiple of 16), nsrc in 1..63,
 * `ctas` CTAs (512 threads each, three tiles of loads in flight per thread, for up to 7 inbox operands and fewer than 128
 * CTAs; 1024 threads otherwise).  Device pointers aligned to the element size; out may equal local. */
hoccl_result_t hoccl_chain_launch(const void* first, size_t stride_bytes, int nsrc, const void* local, void* out, size_t count,
                                  hoccl_dtype_t dtype, int ctas, hoccl_stream_t stream);
/*
 * "SMs used", counted rather than inferred (the paper's Table 1 counts the SMs that communication kernels occupy):
 * launches the SUM kernel (kind 0: out = a + b over bytes / sizeof(dtype) elements) or the copy kernel (kind 1:
 * out <- a, b ignored) with `ctas` CTAs, and every CTA additionally stores the id of the SM it runs on (%smid) to
 * smid_out[block index], a device array of `ctas` 32-bit words.  The number of distinct values is the number of SMs
 * the launch occupied.  Same kernels and launch shapes as the collectives use.
 */
hoccl_result_t hoccl_kernel_sms(int kind, const void* a, const void* b, void* out, size_t bytes, hoccl_dtype_t dtype, int ctas,
                                unsigned int* smid_out, hoccl_stream_t stream);
/*
 * Memory-port probe behind the 8-SM ceiling quoted for the SUM: `ctas` CTAs of 1024 threads only read (mode 0) or only
 * write (mode 1) the device buffer `buf` (16-byte aligned, at least 128 KiB; whole 128 KiB tiles are walked) with 16-byte
 * accesses, 8 in flight per thread.  `sink` is a device word the read mode may write once.  Timed by the caller; together
 * with hoccl_copy_launch (1 read : 1 write) and hoccl_sum_launch (2 : 1) it gives what one SM's memory port carries.
 */
hoccl_result_t hoccl_port_probe(int mode, void* buf, size_t bytes, int ctas, unsigned int* sink, hoccl_stream_t stream);
/*
 * Host only (no device needed): the flattened view the host passes to a batched SUM (kind 0) or copy (kind 1) launch for
 * `nseg` segments given by their ADDRESSES as integers (a, b, out; b unused for the copy) and lengths (elements for the
 * SUM, bytes for the copy) under the kernel shape that `ctas` selects.  Per segment: head (element-wise items before the
 * 16-byte vector body), nvec (vectors in the body), and the running totals of tiles and of element-wise items;
 * *tile_vectors is the tile size in vectors.  The kernels trust this view for every address they form, so tests check its
 * invariants on the CPU: nothing is read or written.
 */
hoccl_result_t hoccl_flatten_inspect(int kind, hoccl_dtype_t dtype, int ctas, int nseg, const uint64_t* a_addr, const uint64_t* b_addr,
                                     const uint64_t* out_addr, const uint64_t* len, uint64_t* tiles_end, uint64_t* scalars_end,
                                     uint64_t* nvec, uint32_t* head, uint64_t* tile_vectors);
/*
 * Host only (no device needed): how a group of `n` moves, given by their ADDRESSES as integers (src[i] -> dst[i], len[i]
 * bytes), is packed into fan-out launches.  Moves with the same source, length and 16-byte phase of the destination share
 * one segment (one read, one store per destination); a launch carries at most 32 segments and 256 destinations.
 * Output, one entry per segment in launch order (arrays of capacity seg_cap): its launch index, source, length, number
 * of destinations, head / nvec of its split under the kernel shape `ctas` selects; its destinations follow each other in
 * dst_out (capacity n).  *n_seg = 0 means no source repeats: the moves go as plain copies.  Nothing is read or written.
 */
hoccl_result_t hoccl_fanout_inspect(int n, const uint64_t* src, const uint64_t* dst, const uint64_t* len, int ctas, int seg_cap,
                                    int* seg_launch, uint64_t* seg_src, uint64_t* seg_len, int* seg_ndst, uint32_t* seg_head,
                                    uint64_t* seg_nvec, uint64_t* dst_out, int* n_seg, int* n_launch);
/*
 * Self-test of the arithmetic: the chain sum of the direct reduce-scatter adds bf16 operands with the native packed add
 * (add.rn.bf16x2); this call compares it on the device with the reference add of every SUM (binary32 add of the widened
 * operands, rounded to nearest even into bf16) for ALL 2^32 pairs of bf16 bit patterns.  counts: DEVICE array of two 64-bit
 * words, zeroed by the caller; after the stream has run it holds {pairs whose results differ, pairs where both results are
 * NaN with different payloads}.  Both must be 0.
 */
hoccl_result_t hoccl_selftest_bf16_add(unsigned long long* counts, hoccl_stream_t stream);

/* ---------------------------------------------------------------- self-tests ------------------- */

/*
 * Failure-detection self-test of the "fused" kernel's bounded waits, without faulting the GPU: enqueues the
 * whole-collective kernel with two copy phases (first and second half of `bytes`, src -> dst, device pointers, bytes a
 * multiple of 32) separated by a grid barrier that waits for one arrival more than the grid delivers.  Every CTA polls
 * for its bounded number of rounds (a second or two), gives up, the kernel ends by itself, the second half is NOT
 * copied, and hoccl_comm_async_error then reports HOCCL_ERR_TIMEOUT; the barrier words are clean for the next call.
 */
hoccl_result_t hoccl_selftest_barrier_timeout(hoccl_comm_t comm, void* dst, const void* src, size_t bytes, hoccl_stream_t stream);

/*
 * The same for the bounded waits of the "roles" kernel (communicator parameter "roles" = 1, else HOCCL_ERR_UNSUPPORTED):
 * enqueues the all-reduce the arguments describe (as hoccl_allreduce) with summing CTAs that wait for one mover more than
 * the grid has.  They poll for their bounded number of rounds (a second or two) and give up, every other CTA sees the
 * give-up flag and leaves, the kernel ends by itself (the receive buffers are then NOT the all-reduce), and
 * hoccl_comm_async_error reports HOCCL_ERR_TIMEOUT; the counters are clean for the next call.
 */
hoccl_result_t hoccl_selftest_roles_timeout(const void* const* sendbufs, void* const* recvbufs, size_t count, hoccl_dtype_t dtype,
                                            hoccl_comm_t comm, hoccl_stream_t stream);

/* ---------------------------------------------------------------- plan inspection (host only) --- */

/*
 * The planner (paper Sec. 3.4: a collective becomes stages of point-to-point flows that are cut into
 * chunks for the copy queue) is pure host code; these calls expose its output so that it can be
 * checked without a GPU.  Addresses in a plan are byte offsets: buffer kinds below say what they are
 * relative to.
 */
typedef enum { HOCCL_PLAN_ALLREDUCE = 0, HOCCL_PLAN_REDUCE_SCATTER = 1, HOCCL_PLAN_ALLGATHER = 2, HOCCL_PLAN_ALLTOALL = 3,
               HOCCL_PLAN_ALLREDUCE_FWD = 4, HOCCL_PLAN_REDUCE_SCATTER_FWD = 5, /* the "forward" variants */
               HOCCL_PLAN_ALLREDUCE_AGD = 6, HOCCL_PLAN_ALLGATHER_DIRECT = 7,   /* the "ag_direct" variants */
               HOCCL_PLAN_ALLREDUCE_FWD_AGD = 8 /* both */ } hoccl_plan_kind_t;
/* General form: a base kind (0..3) OR-ed with flags; the numbered variants above are shorthands. */
typedef enum { HOCCL_PLAN_FLAG_FORWARD = 16, HOCCL_PLAN_FLAG_AG_DIRECT = 32, HOCCL_PLAN_FLAG_RS_DIRECT = 64 /* "rs_direct" */,
               HOCCL_PLAN_FLAG_GRADED = 128 /* "piece_grade": smaller first and last pieces */ } hoccl_plan_flag_t;
/* CHAIN: out = (((s_0 + s_1) + ...) + s_{nsrc-1}) + local, every add rounded into the I/O dtype; s_j at src_off + j * src_stride */
typedef enum { HOCCL_OP_MOVE = 0, HOCCL_OP_SUM = 1, HOCCL_OP_CHAIN = 2 } hoccl_plan_op_kind_t;
typedef enum { HOCCL_BUF_SEND = 0, HOCCL_BUF_RECV = 1, HOCCL_BUF_INBOX = 2, HOCCL_BUF_PARTIAL = 3 } hoccl_buf_kind_t;

typedef struct {
  int kind;      /* hoccl_plan_op_kind_t */
  int phase;     /* 0 reduce-scatter, 1 all-gather, 2 own-chunk / own-block copy, 3 all-to-all stage */
  int step;      /* ring step s (all-to-all: stage k, destination = rank + k; direct all-gather: stage k - 1) */
  int piece;     /* pipeline piece index */
  int rank;      /* MOVE: source rank; SUM: the rank that sums */
  int dst_rank;  /* MOVE: destination rank; SUM: same as rank (forward variants: the rank whose slot receives the result) */
  int chunk;     /* ring chunk index */
  int src_buf, dst_buf, local_buf; /* hoccl_buf_kind_t; local_buf only for SUM */
  uint64_t src_off, dst_off, local_off; /* byte offsets from the start of those buffers (scratch: from the start of the rank's slot) */
  uint64_t bytes;
  int group;     /* ops of one group are issued together (one batched kernel launch or R copies) */
  int nsrc;      /* CHAIN: number of inbox operands (R-1); 1 otherwise */
  uint64_t src_stride; /* CHAIN: bytes between consecutive inbox operands (one scratch slot) */
} hoccl_plan_op_t;

typedef struct hoccl_plan* hoccl_plan_t;

/* Builds the plan for `kind` over R ranks.  `count` as in the collective; in_place as defined at the top of
 * this file; piece_bytes / max_pieces as the parameters of the same name.  send_align: HOST array of R bytes,
 * the low 4 bits of each rank's send pointer (NULL = all 16-byte aligned); it only decides where inside its
 * scratch region a piece is placed so that SUM operands share their 16-byte phase.  Free with hoccl_plan_destroy. */
hoccl_result_t hoccl_plan_build(hoccl_plan_t* plan, int kind, int R, size_t count, hoccl_dtype_t dtype, int in_place,
                                size_t piece_bytes, int max_pieces, const unsigned char* send_align);
/* Bytes of one rank's scratch slot (inbox or partial) under this plan.  Rank r's inbox is hoccl_plan_inbox_slots slots at
 * r * slots * slot bytes (1 slot; R-1 for the direct reduce-scatter); the partial slots, one per rank, follow all inboxes. */
size_t hoccl_plan_slot_bytes(hoccl_plan_t plan);
int hoccl_plan_inbox_slots(hoccl_plan_t plan);
/* Scratch bytes a call with this plan needs. */
size_t hoccl_plan_scratch_bytes(hoccl_plan_t plan);
void hoccl_plan_destroy(hoccl_plan_t plan);
int hoccl_plan_num_ops(hoccl_plan_t plan);
int hoccl_plan_num_groups(hoccl_plan_t plan);
hoccl_result_t hoccl_plan_get_op(hoccl_plan_t plan, int index, hoccl_plan_op_t* out);
/* Dependencies are between groups: writes up to `cap` predecessor group ids of `group` into deps, returns their number. */
int hoccl_plan_group_deps(hoccl_plan_t plan, int group, int* deps, int cap);

/* ---------------------------------------------------------------- option rules (host only) ---- */

/*
 * How a communicator's settings combine for one call, without a device: the schedule (base collective OR-ed with
 * hoccl_plan_flag_t bits), the executor and the move route the call would run on, or HOCCL_ERR_UNSUPPORTED when what was
 * asked for does not fit together.  hoccl_comm_set_param in hoccl.h states the rules; every entry point applies exactly
 * this function, so a combination is either served as asked or refused, never changed silently.
 * kind: 0 all-reduce, 1 reduce-scatter, 2 all-gather, 3 all-to-all; count in that collective's convention; the option
 * fields carry the values of the parameters of the same name; scratch_bytes = attached scratch (0: none); host_call = 1
 * for hoccl_host_allreduce.  (HOCCL_PLAN_FLAG_GRADED is not part of the answer: a call adds it by message size, "piece_grade".)
 */
typedef struct {
  int kind, R;
  size_t count;
  int dtype, path;
  long onepass, forward, fused, rs_direct, ag_direct, handshake, use_graph, ce_small_bytes, ce_small_ctas, copy_ctas;
  size_t scratch_bytes;
  int host_call;
  long roles;
} hoccl_options_t;
typedef enum { HOCCL_EXEC_GRAPH = 0, HOCCL_EXEC_STREAMS = 1, HOCCL_EXEC_ONE_KERNEL = 2, HOCCL_EXEC_ONEPASS = 3, HOCCL_EXEC_PROXY = 4,
               HOCCL_EXEC_ROLES = 5 } hoccl_executor_t;
typedef struct {
  int plan_kind;    /* base collective | hoccl_plan_flag_t bits: what hoccl_plan_build is given */
  int executor;     /* hoccl_executor_t */
  int path;         /* the route the moves take (HOCCL_PATH_SM for a small message on HOCCL_PATH_CE) */
  long copy_ctas;   /* CTAs of its copy launches */
  int small_switch; /* 1 if the small-message rule ("ce_small_bytes") changed the route */
} hoccl_resolved_t;
hoccl_result_t hoccl_options_resolve(const hoccl_options_t* options, hoccl_resolved_t* out);

#ifdef __cplusplus
}
#endif
#endif /* HOCCL_DIAG_H_ */
