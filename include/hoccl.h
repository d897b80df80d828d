/*
 * hoccl.h - C ABI of libhoccl.so: ring collectives and point-to-point transfers over R logical
 * ranks that live as R disjoint buffers in the HBM of ONE B200.
 *
 * Background.  HOCCL (the paper) runs collectives as host-issued chunked transfer schedules so that
 * data movement leaves the SMs free (Sec. 3.1 "Overview": stream manager, point-to-point executor,
 * collective scheduler).  This library builds the data-parallel hot path of that method for one
 * GPU: a collective is planned on the host as a DAG of chunk MOVEs and, for reductions, per-step
 * chunk SUMs; every MOVE is a plain device-to-device copy (driver copy route, or an SM copy kernel
 * with a CTA budget as the comparison path); the SUM is a hand-written sm_100a kernel limited to a
 * small CTA budget.  The paper leaves reductions out of scope (Sec. 4 "Limitations"); the ring
 * reduce-scatter here is the textbook one in a fixed order, stated next to hoccl_allreduce.
 *
 * Conventions that hold for every entry point unless stated otherwise
 *  - Pointers named `send`/`recv` are HOST arrays of R DEVICE pointers: send[r] is rank r's input
 *    buffer X_r, recv[r] its output buffer Y_r.  The arrays are read during the call and not kept.
 *    All device buffers belong to the caller and live on the communicator's device.
 *  - `count` is in elements of `dtype`, NCCL style (the paper's runtime extends NCCL and is measured
 *    with nccl-tests, Sec. 5 "Testbed"): see each collective.
 *  - Calls are asynchronous: they enqueue work and return.  The work starts after everything
 *    enqueued earlier on `stream` and everything enqueued later on `stream` sees it complete: the
 *    paper's operator-level temporal ordering (abstract; Sec. 3.2 "Stream Manager").  No call
 *    synchronises the host with the device, except where a call says so.
 *  - Errors are return codes; nothing is enqueued when a call fails with an argument error.
 *    count == 0 is HOCCL_OK and enqueues nothing.  X_r is never written (unless it aliases Y_r).
 *  - Buffers of different ranks must not overlap.  In place is legal: allreduce with
 *    send[r] == recv[r]; reduce_scatter with recv[r] == send[r] + r*count; allgather with
 *    send[r] == recv[r] + r*count (element offsets).
 *  - One host thread per communicator.  Device memory is the caller's: scratch and staging are
 *    attached with hoccl_comm_set_scratch / hoccl_comm_set_staging.  The two exceptions are stated where
 *    they apply: handshake mode allocates 512 bytes once, and hoccl_allreduce_static uses a fixed array
 *    that is part of the library image.
 *  - Probes, self-tests, direct kernel launches and plan inspection are declared in hoccl_diag.h.
 *  - The CUDA device must be present: every entry point that touches the device returns
 *    HOCCL_ERR_CUDA otherwise.  There is no CPU fallback.
 */
#ifndef HOCCL_H_
#define HOCCL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hoccl_comm* hoccl_comm_t;
/* a CUDA stream handle (cudaStream_t / CUstream) passed as an opaque pointer; NULL is the legacy default stream */
typedef void* hoccl_stream_t;

typedef enum {
  HOCCL_OK = 0,
  HOCCL_ERR_INVALID_ARG = 1, /* null pointer, rank or R out of range, src == dst, overlapping rank buffers, misaligned pointer */
  HOCCL_ERR_UNSUPPORTED = 2, /* op other than sum, unknown dtype, unknown parameter key */
  HOCCL_ERR_CUDA = 3,        /* a CUDA call failed (no device, bad stream, ...) */
  HOCCL_ERR_MISMATCH = 4,    /* send/recv matched with different count or dtype; the parked post is dropped */
  HOCCL_ERR_PENDING = 5,     /* destroy with unmatched send/recv posts */
  HOCCL_ERR_SCRATCH = 6,     /* scratch or staging memory missing or too small */
  HOCCL_ERR_INTERNAL = 7,
  HOCCL_ERR_TIMEOUT = 8      /* handshake mode: the watchdog released a stream (asynchronous, see hoccl_comm_async_error) */
} hoccl_result_t;

typedef enum { HOCCL_FLOAT32 = 0, HOCCL_BFLOAT16 = 1 } hoccl_dtype_t;
typedef enum { HOCCL_SUM = 0 } hoccl_op_t;

/*
 * How MOVEs are carried out.
 *  HOCCL_PATH_CE : one device-to-device cudaMemcpyAsync (or memcpy graph node) per move.  This is
 *                  the copy-engine route of the paper (Sec. 2.3 "DMA Engines", Sec. 3.3): between two
 *                  GPUs the driver services it with a DMA engine and no SM.  Whether a copy inside ONE
 *                  device is also SM free is up to the driver; hoccl_probe_move_needs_sm measures it.
 *  HOCCL_PATH_CE_HOST : every move is a device-to-host copy into PINNED host staging followed by a host-to-device
 *                  copy out of it.  Both legs are served by the copy engines (Sec. 2.3), so this is the one route
 *                  on a single device that really occupies no SM (hoccl_probe_move_needs_sm confirms it); the price
 *                  is PCIe bandwidth.  Needs hoccl_comm_set_host_staging with room for every move of a call
 *                  (all-reduce: 2 * S * (R-1) bytes plus 256 per move; send/recv: the message).  A send/recv message
 *                  larger than one chunk ("piece_bytes", at least 1 MiB) is pipelined through the staging area chunk by
 *                  chunk, the outbound leg of chunk k+1 beside the inbound leg of chunk k (Sec. 3.3.1).  Not available
 *                  for hoccl_alltoallv or in handshake mode.
 *  HOCCL_PATH_SM : the comparison baseline (the paper's "NCCL with an SM budget", Sec. 5 "Baselines"):
 *                  all moves of a step run in one launch of an SM copy kernel with `copy_ctas` CTAs.
 */
typedef enum { HOCCL_PATH_CE = 0, HOCCL_PATH_SM = 1, HOCCL_PATH_CE_HOST = 2 } hoccl_path_t;

typedef struct {
  double host_launch_us; /* host time spent inside the last collective / matched p2p call (paper Sec. 5 "CPU launch overhead") */
  long n_moves;          /* MOVE operations of the last call (copies on the CE path, segments on the SM path) */
  long n_move_launches;  /* SM copy kernel launches of the last call (0 on the CE path) */
  long n_sum_launches;   /* SUM kernel launches of the last call */
  long max_sum_ctas;     /* CTAs of the widest SUM launch */
  long max_copy_ctas;    /* CTAs of the widest SM copy launch */
  long n_pieces;         /* pipeline pieces per ring chunk */
  long graph_hit;        /* 1 if the call replayed a cached CUDA graph, 0 if it built one or used streams */
  double sum_kernel_ms;  /* with parameter "profile" = 1: total device time of SUM launches since hoccl_profile_reset */
  long sum_kernel_launches_timed;
  double sum_kernel_bytes; /* algorithmic bytes (2 reads + 1 write per element) of those launches */
  double copy_kernel_ms;   /* the same for copy_kernel launches (SM path, graph executor) */
  long copy_kernel_launches_timed;
  double copy_kernel_bytes; /* algorithmic bytes (1 read + 1 write per byte) of those launches */
  long n_order_launches;    /* empty one-warp kernels of the last call that only order copy nodes inside its graph (copy routes) */
} hoccl_stats_t;

/* ---------------------------------------------------------------- communicator ----------------- */

/*
 * Creates a communicator of R logical ranks (1 <= R <= 64) on CUDA device `device`: internal
 * streams and events only, no device memory.  Errors: INVALID_ARG (comm NULL, R out of range),
 * CUDA (no such device).
 */
hoccl_result_t hoccl_comm_init(hoccl_comm_t* comm, int R, int device);

/* Frees host state, streams, events and cached graphs.  Synchronises the internal streams.
 * HOCCL_ERR_PENDING (and nothing freed) if unmatched send/recv posts remain.
 * Handshake mode: hand-overs that are still open after one watchdog period (a stream that has not reached its call yet
 * because it is busy with earlier work, a schedule that has not finished) are released by force, so that no stream
 * waits on a communicator that is gone: such a stream goes on WITHOUT the result of that call, everything is freed as
 * usual, and the call returns HOCCL_ERR_TIMEOUT to say so.  (The few hundred bytes of pinned counters stay allocated
 * for the life of the process in that case: the late stream still reads them when it gets there.) */
hoccl_result_t hoccl_comm_destroy(hoccl_comm_t comm);

/* Upper bound of the scratch bytes any collective needs for up to `max_count` elements of `dtype`
 * per rank buffer (allreduce convention) with R ranks: per rank one inbox and one partial slot of
 * one ring chunk each, padded.  0 for R == 1. */
size_t hoccl_scratch_bytes(int R, size_t max_count, hoccl_dtype_t dtype);
/* The same bound with the "rs_direct" parameter set: per rank R-1 inbox slots of one ring chunk each, padded.  It also covers
 * every call without that parameter when R >= 3. */
size_t hoccl_scratch_bytes_direct(int R, size_t max_count, hoccl_dtype_t dtype);

/* Attaches caller-owned device scratch (256-byte aligned).  Reductions need it; all-gather and p2p do
 * not.  Contents are undefined between calls.  Collectives that overlap in time on different streams
 * must not share a communicator. */
hoccl_result_t hoccl_comm_set_scratch(hoccl_comm_t comm, void* dev_ptr, size_t bytes);

/* Attaches caller-owned device staging memory used only by the hoccl_host_* entry points. */
hoccl_result_t hoccl_comm_set_staging(hoccl_comm_t comm, void* dev_ptr, size_t bytes);

/* Attaches caller-owned PINNED host memory (cudaHostAlloc / cudaHostRegister) used by HOCCL_PATH_CE_HOST.
 * INVALID_ARG if the pointer is not page-locked host memory. */
hoccl_result_t hoccl_comm_set_host_staging(hoccl_comm_t comm, void* pinned_host_ptr, size_t bytes);

hoccl_result_t hoccl_comm_set_path(hoccl_comm_t comm, hoccl_path_t path);

/*
 * Tuning and diagnostics.  Keys:
 *  "sum_ctas"    CTAs of a SUM launch, 1..1024 (default 8: the SM budget for sums)
 *  "copy_ctas"   CTAs of an SM copy launch, 1..1024 (default 8)
 *  "piece_bytes" pipeline piece size in bytes (rounded to a multiple of 1024).  If the key is not set: for reductions, whole
 *                ring chunks (up to 256 MiB) on HOCCL_PATH_CE and on HOCCL_PATH_SM when both CTA budgets are 128 or more (pieces exist to overlap one
 *                piece's move with another piece's sum, which neither driver copies nor whole-GPU grids do); otherwise
 *                4 MiB, and on the SM path with CTA budgets below 64 a reduction whose ring chunk is 1 MiB or more is
 *                cut into at least two pieces so that one piece's copy kernel overlaps the other's sum kernel.
 *  "max_pieces"  cap on pieces per ring chunk (default 8)
 *  "lanes"       internal move streams of the stream executor, 1..8 (default 4)
 *  "p2p_split"   a send/recv message of 32 MiB or more on the CE path is cut into up to this many slices that
 *                run on different lanes, 1..8 (default 1 = one copy per message; measured: slices do not help
 *                on one device because every driver copy already spreads over the whole GPU)
 *  "ce_sub_bytes" graph executor, CE path: a move between this many bytes and 16 MiB is issued as sub-copies of
 *                this size (0 = off, the default; measured: no gain once a graph's first copies share one predecessor)
 *  "onepass"     1 = all-reduce and reduce-scatter run as ONE kernel ("sum_ctas" CTAs) that reduces every element in
 *                registers in the ring's order and rounding and writes it to its destinations: the same bits, R reads
 *                + R (or 1) writes per element instead of 7(R-1) bytes per wire byte, no moves, no scratch.  It is not
 *                rank local (one kernel reads every rank's buffer), so it only makes sense on one device and is kept
 *                as the comparison point that shows what the rank-local schedule costs.  0 = off (default).
 *  "forward"     1 = fused sum-and-forward variant of the ring reduce-scatter: the SUM of step s writes its result
 *                straight into the next rank's inbox, so only step 0 needs moves (3 instead of 5 bytes of traffic per
 *                wire byte in that phase).  Same bits.  A SUM then stores into another rank's memory, as SM-driven
 *                libraries do: it is the second comparison point for what rank locality costs.  0 = off (default).
 *  "ag_direct"   1 = the all-gather (alone or as the second half of an all-reduce) runs as the stage decomposition of its
 *                traffic matrix (paper Sec. 3.4): every rank sends its own final chunk to every other rank, R-1
 *                contention-free permutation stages r -> r+k that depend only on the chunk being final, instead of R-1
 *                ring hops that each wait for the previous one.  Rank local (a rank sends what it owns), same bytes
 *                moved, same bits; the moves of all stages can be in flight together.  HOCCL_PATH_SM: one batched launch
 *                in which every chunk is read once and stored R-1 times (S R instead of 2 S (R-1) bytes of traffic);
 *                HOCCL_PATH_CE_HOST: a chunk goes out to the host staging once and comes back R-1 times.
 *                0 = the ring all-gather.  2 (default) = automatic: direct where it was measured faster on B200 (always on
 *                HOCCL_PATH_SM and HOCCL_PATH_CE_HOST; on HOCCL_PATH_CE while a ring chunk is at most 64 MiB), ring elsewhere.
 *  "rs_direct"   1 = the reduce-scatter (alone or as the first half of an all-reduce) runs as the stage decomposition of its
 *                traffic matrix (paper Sec. 3.4: rank r owes its contribution to chunk d to rank d): R-1 contention-free
 *                permutation stages r -> r+k that wait for nothing, into R-1 inbox slots of the owner, and then ONE sum
 *                per rank that adds the R-1 arrived contributions and its own in the ring's order, rounding into the I/O
 *                dtype after every add (the chain sum, "sum_ctas" CTAs).  Rank local, the ring's bits; every output byte is
 *                written once instead of R-1 times: 2 S (R-1) + S (R+1) bytes of traffic instead of 5 S (R-1), and under
 *                an SM budget, where a sum is bound by the SMs' memory ports, R reads + 1 write per output instead of
 *                (R-1) x (2 reads + 1 write).  Needs hoccl_scratch_bytes_direct bytes of scratch (R-1 slots per rank
 *                instead of 2); with less the call returns HOCCL_ERR_SCRATCH.  0 = the ring reduce-scatter, step by step.
 *                2 (default) = automatic: direct whenever the attached scratch is large enough for it and neither "forward",
 *                "fused" nor "onepass" is set (it was measured faster than the ring at every size and on every path), the ring
 *                otherwise.  So a communicator with hoccl_scratch_bytes of scratch runs the ring, one with
 *                hoccl_scratch_bytes_direct runs the direct form; the bits are the same.
 *  "ce_small_bytes" on HOCCL_PATH_CE a call whose per-rank message (S in the convention of each collective: all-reduce
 *                count, reduce-scatter / all-gather / all-to-all R * count elements) is at most this many bytes issues its
 *                moves as batched launches of the SM copy kernel with "ce_small_ctas" CTAs instead of driver copies, i.e.
 *                it runs on the route of HOCCL_PATH_SM (hoccl_last_stats shows the launches).  Inside one device a driver
 *                copy spares no SM (hoccl_probe_move_needs_sm) and takes microseconds to start, so below a crossover the
 *                kernel is a pure gain: measured on B200 with the default schedule and 8-CTA sums, R = 8 bf16 all-reduce of
 *                4 KiB 34 -> 10 us, 1 MiB 48 -> 25 us, 4 MiB 88 -> 54 us, 8 MiB 107 -> 97 us, equal from 16 MiB on; R = 4 fp32
 *                all-reduce of 4 MiB 37 -> 33 us.  Default 8 MiB; 0 = driver copies at every size.  "HOCCL_PATH_CE" therefore
 *                means: the copy route above this size.  Not applied to hoccl_host_allreduce, send/recv or hoccl_alltoallv.
 *  "ce_overlap"  HOCCL_PATH_CE, direct reduce-scatter: the ring chunks are cut into this many pieces and every piece's three
 *                parts (the reduce-scatter's moves, the chain sum, the all-gather's moves) become graphs of their own that
 *                run on three internal streams, ordered by events, so that one piece's driver copies run beside another
 *                piece's sum (inside ONE graph, and on plain streams, they were never seen to overlap).  Sums still run one
 *                at a time.  Costs ~8 us of host time per piece and call.  -1 (default) = automatic: 2 pieces from 2 MiB per
 *                ring chunk, from 4 MiB on pieces of about 4 MiB (at least 4, at most 32 of them), off below; 0 = off;
 *                2..64 = that many pieces.  Ignored when "piece_bytes" is set.
 *  "ce_small_ctas" CTAs of those launches, 1..1024 (default 148: like the driver's own copies they may use the whole GPU,
 *                for tens of microseconds)
 *  "order_kernels" 1 (default) = on the copy routes the graph executor puts an empty one-warp kernel in front of a graph's
 *                first copies and behind every group of copies that other copies (or the end of the graph) wait for.
 *                Measured on B200: a copy node that waits for earlier stream work or for several copy nodes starts ~4 us
 *                late per node, and a GEMM on another stream loses half of its throughput beside such graphs (54 %
 *                against 8 % for the gradient bucket).  0 = plain graphs (the comparison point).
 *  "fused"       1 = on HOCCL_PATH_SM the whole collective runs as ONE cooperative kernel that walks the ring steps with a
 *                grid-wide barrier between dependent steps (how an SM-driven library runs a collective: the paper's
 *                "NCCL under an SM budget" baseline, Sec. 5).  The schedule stays rank local and the bits are the same.
 *                Its grid is min(sum_ctas, copy_ctas) CTAs (copy_ctas for pure moves), fewer for small messages.
 *                Measured on B200 (R = 8, bf16, whole GPU): a grid barrier costs ~4 us against ~1.5 us for a kernel
 *                boundary inside a CUDA graph, so below 128 MiB per rank the graph of per-step kernels is faster (4 KiB
 *                all-reduce: 31 against 96 us); from 128 MiB on the one-kernel form is 1-3 % faster (no ramp and tail
 *                per step: 0.78-0.80 against 0.76-0.78 of the 8 TB/s roofline).  Under an 8-CTA budget the graph is
 *                faster at every size, because it overlaps a copy kernel with a sum kernel.
 *                Every barrier wait is bounded; a wait that runs out ends the kernel and is reported by
 *                hoccl_comm_async_error as HOCCL_ERR_TIMEOUT.  The library allocates 16 bytes of device memory and 4 bytes
 *                of pinned host memory of its own on first use (the third exception to "device memory is the caller's").
 *                Refused on the other paths and in handshake mode (see the rules below); plans too large for one launch (more
 *                than 480 chunk operations or 96 steps: an all-reduce beyond 12 ranks) run as a graph.  0 = off (default).
 *  "roles"       1 = on HOCCL_PATH_SM all-reduce and reduce-scatter calls of 2 to 8 ranks run the stage-decomposed schedule
 *                ("rs_direct", "ag_direct") as ONE cooperative kernel whose CTAs have roles: the first min(sum_ctas, 64) CTAs
 *                only sum, copy_ctas further CTAs only move, and the pieces of a chunk are pipelined between them through
 *                counters in device memory (moves of piece p + 1 run beside the sums of piece p; paper Sec. 3.3, chunk
 *                pipelining, without a launch per piece and kernel).  Rank local, same bits.  Measured on B200 (R = 8, bf16,
 *                8 + 40 CTAs) it equals the graph of kernels with the same budgets within a few per cent (40 MiB per rank
 *                0.377 against 0.380 ms, 256 MiB 2.28 against 2.32 ms).  It needs the scratch of the direct form
 *                (hoccl_scratch_bytes_direct; HOCCL_ERR_SCRATCH otherwise).  Every wait is bounded; a wait that runs out ends
 *                the kernel and is reported by hoccl_comm_async_error as HOCCL_ERR_TIMEOUT.  The library allocates 1 KiB of
 *                device memory and 4 bytes of pinned host memory per communicator on first use, and per cached call
 *                signature a table of at most 200 KiB in device memory (further exceptions to "device memory is the
 *                caller's").  When sum_ctas + copy_ctas CTAs cannot be resident together, or the tables of a call's pieces
 *                exceed 200 KiB (more than ~40 pieces at 8 ranks), the same plan runs as a graph.  Other calls ignore the
 *                setting.  0 = off (default).
 *  "piece_grade" all-reduce and reduce-scatter on the stage-decomposed schedule: 1 = the pieces of a ring chunk are graded, the
 *                first and the last ones smaller (a third, two thirds of a middle piece; pieces of 256 KiB or more only), so that
 *                less of the moves in front of the first sum and behind the last one is exposed; 0 = equal pieces; -1 (default)
 *                = automatic: graded from 8 MiB per ring chunk on under a SUM budget (sum_ctas < 64), where it was measured to
 *                gain 1-5 %, equal otherwise (below that size the small outer pieces cost more than they save).  Same
 *                operations, same bits.
 *  "host_pieces" pieces per ring chunk of the pipelined hoccl_host_allreduce (1..64, default 8; 1 = not pipelined)
 *  "use_graph"   1 = run a cached CUDA graph built from the plan (default), 0 = streams and events
 *  "handshake"   1 = the paper's stream manager (Sec. 3.2): instead of launching into the caller's stream, the call
 *                enqueues three stream memory operations (write "hand-over n has arrived", wait for "hand-over n is
 *                released", write "hand-over n is behind me"; the counters live in pinned host memory and only grow) and
 *                hands the schedule to a CPU proxy thread that polls the counters, runs the schedule on an internal stream
 *                and then releases the caller's stream.  send/recv posts are matched by the proxy AFTER each stream has reached its post, so a
 *                post may wait for a partner that is posted later (the paper's semantics, Sec. 3.3.2); count/dtype
 *                mismatches and unmatched posts are then reported asynchronously (hoccl_comm_async_error).
 *                0 = off (default).  Results are identical bit for bit.  Handshake mode needs HOCCL_PATH_SM: calls on
 *                the other paths return HOCCL_ERR_UNSUPPORTED, because on one device a driver copy issued by the proxy
 *                can queue up behind copies that the parked stream itself has waiting and then never start.
 *                The two sides of a send/recv must be
 *                posted on different streams (a stream parked in its own post cannot reach the partner's).  The
 *                first use creates the proxy: a thread, pinned host memory for 64 sets of counters and 512 bytes of
 *                device memory (one of the library's own device allocations stated in this header), and loads every kernel, because
 *                first-use work in the driver must not happen while a stream is parked.
 *  "watchdog_ms" handshake mode: after this long (default 10000) the stream of an unmatched post is released without its
 *                transfer and HOCCL_ERR_TIMEOUT is recorded, so no stream can wait on this library forever
 *  "p2p_strict"  1 = send/recv posts go through the CPU proxy as in handshake mode while collectives are launched directly:
 *                a post then holds its stream at the post until the transfer is done, whichever side posts first (the
 *                paper's semantics, Sec. 3.3.2), instead of parking on the host (see hoccl_send).  Needs HOCCL_PATH_SM,
 *                like handshake mode.  0 = off (default).
 *  "model_gpus_per_node"  hoccl_alltoallv only: 0 (default) or >= R = all ranks in one NVLink domain; g in 1..R-1 = the ranks are
 *                modelled as nodes of g GPUs each and inter-node flows take the forwarding copies and the RDMA leg of the
 *                paper's scheduler as real copies through the staging memory (see hoccl_alltoallv)
 *  "model_rdma_sub_bytes" modelled topology: the RDMA leg of a chunk is issued in sub-copies of this many bytes, one after the
 *                other, as a NIC serialises its queue (0 = one copy per chunk, default)
 *  "profile"     1 = time every SUM launch with CUDA events; read the totals with hoccl_last_stats after
 *                synchronising (with graphs only the latest replay of each cached graph is readable, so
 *                read after every step)
 * How the settings combine (one rule set, applied by every collective before it plans; hoccl_options_resolve in
 * hoccl_diag.h evaluates it without a device).  A value of 1 asks for something, 2 is automatic and yields to whatever was
 * asked for; a combination that does not fit together makes the CALL return HOCCL_ERR_UNSUPPORTED with nothing enqueued,
 * it is never changed silently:
 *   - "handshake" needs HOCCL_PATH_SM and cannot be combined with "onepass" or "fused" (the proxy replays graphs);
 *   - "fused" is an executor of HOCCL_PATH_SM: refused on the other paths; refused with "rs_direct" = 1 (the one-kernel
 *     form has no chain phase); it ignores "use_graph" and is not used by hoccl_host_allreduce; plans beyond its capacity
 *     (see "fused") run as a graph;
 *   - "roles" applies to all-reduce and reduce-scatter calls (hoccl_host_allreduce excepted) and runs the direct schedule
 *     on HOCCL_PATH_SM: refused on the other paths, for fewer than 2 or more than 8 ranks, and together with "handshake",
 *     "onepass", "forward", "fused", "rs_direct" = 0 or (all-reduce) "ag_direct" = 0; it ignores "use_graph";
 *   - "onepass" applies to all-reduce and reduce-scatter calls, ignores the path, and for those calls is refused together
 *     with "forward", "fused", "rs_direct" = 1 or (all-reduce) "ag_direct" = 1; other collectives ignore it;
 *   - "forward" applies to all-reduce and reduce-scatter calls and is refused with "rs_direct" = 1;
 *   - "use_graph" chooses between graph replay and the stream executor where neither "handshake" nor "fused" decides.
 * None of them changes a single result bit.  Errors of set_param itself: UNSUPPORTED (unknown key), INVALID_ARG (range).
 */
hoccl_result_t hoccl_comm_set_param(hoccl_comm_t comm, const char* key, long value);
hoccl_result_t hoccl_comm_get_param(hoccl_comm_t comm, const char* key, long* value);

/* ---------------------------------------------------------------- collectives ------------------ */

/*
 * Ring all-reduce (sum) = ring reduce-scatter followed by ring all-gather.
 * send[r], recv[r]: `count` elements each.  After completion every recv[r] holds the same vector.
 *
 * Order of the sum (fixed; results are bit-reproducible).  The buffer is cut into R ring chunks of
 * q = ceil(count/R) elements (trailing chunks may be short or empty).  Data travels r -> (r+1) mod R.
 * At step s = 0..R-2 rank r sends chunk (r-1-s) mod R (its own data at s = 0, else the partial it just
 * produced) and then adds what it received to its own chunk (r-2-s) mod R:
 *     out[i] = round_to_dtype( float(received[i]) + float(own[i]) )     one binary32 add, RNE
 * so element i of chunk c ends as ((x_{c+1} + x_{c+2}) + ... + x_{c+R-1}) + x_c (rank indices mod R),
 * and the partial is stored in `dtype` at every hop (bf16 is re-rounded R-1 times).
 * The paper has no reduction (Sec. 4 "Limitations"); moves follow its chunked, pipelined transfer
 * schedule (Sec. 3.3 "chunk pipelining", Sec. 3.4 "Flow-size-aware chunk scheduling").
 * Needs scratch (hoccl_scratch_bytes).  Errors: INVALID_ARG, UNSUPPORTED, SCRATCH, CUDA.
 */
hoccl_result_t hoccl_allreduce(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                               hoccl_op_t op, hoccl_comm_t comm, hoccl_stream_t stream);

/*
 * Ring reduce-scatter (sum).  send[r]: R*count elements; recv[r]: count elements = chunk r of the
 * sum, reduced in the order given above with chunk c = elements [c*count, (c+1)*count).
 * Needs scratch.
 */
hoccl_result_t hoccl_reduce_scatter(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                                    hoccl_op_t op, hoccl_comm_t comm, hoccl_stream_t stream);

/*
 * Ring all-gather (paper Sec. 5 "AllGather": the data-parallel pattern HOCCL targets).
 * send[r]: count elements; recv[r]: R*count elements = send[0] | send[1] | ... | send[R-1].
 * Pure moves: R-1 ring steps, plus the copy of the own chunk when not in place.  No scratch.
 */
hoccl_result_t hoccl_allgather(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                               hoccl_comm_t comm, hoccl_stream_t stream);

/*
 * All-to-all (paper Sec. 5 "All-to-All", its second benchmarked collective).  send[r] and recv[r] hold R blocks
 * of `count` elements; block j of recv[r] becomes block r of send[j].  Pure moves: the R(R-1) remote blocks
 * travel in R-1 permutation stages (stage k: every rank r sends to rank (r+k) mod R: a contention-free matching,
 * the degenerate case of the paper's stage decomposition, Sec. 3.4), plus one copy of the own block.
 * No scratch.  There is no in-place form: send[r] and recv[r] must not overlap (INVALID_ARG otherwise).
 */
hoccl_result_t hoccl_alltoall(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                              hoccl_comm_t comm, hoccl_stream_t stream);

/*
 * User-defined pattern (paper Sec. 3.4: "arbitrary user-defined collective communication patterns" go through the
 * traffic matrix).  MPI-style all-to-allv over the R logical ranks: rank u sends sendcounts[u*R+v] elements, taken
 * from send[u] + sdispls[u*R+v], to rank v, which stores them at recv[v] + rdispls[v*R+u] (counts and
 * displacements are HOST arrays of R*R entries, in elements).  u == v is a local copy.
 * The flows form the origin traffic matrix C; the collective scheduler (hoccl_sched_*) cuts it into stages by
 * peeling matchings (Algorithm 1 with an empty RDMA domain: T = C) and, inside a stage, serves every source rank's
 * flows from one serial queue in a size-weighted chunk interleaving (chunk = the "piece_bytes" parameter, at least
 * 64 KiB; chunks that follow one another in a queue and continue the same flow are issued as one operation).  Stages
 * run one after the other.  With "use_graph" = 1 (default) the schedule becomes a CUDA graph that is cached under the
 * call's full signature (every pointer, count and displacement), so a pattern that repeats on the same buffers replays
 * it; otherwise, and with "use_graph" = 0, it is issued with streams and events.  No scratch.
 * Modelled topology ("model_gpus_per_node" = g with 0 < g < R): the R logical ranks are treated as GPUs of R / g nodes (rank r
 * sits on node r / g, the last node may be smaller) and the scheduler runs the paper's full expansion (Eq. 2-4, Algorithm 1):
 * a flow between two nodes is carried, portion by portion as Algorithm 1 stages it, by a forwarding copy to the sender's
 * symmetric peer, the "RDMA" leg to the receiver's symmetric peer and a forwarding copy to the receiver, all as real copies
 * through the memory attached with hoccl_comm_set_staging, while native flows fill the NVLink slack of the stages.  The
 * received bytes are the same.  Needs staging of at least twice the inter-node bytes of the call, every flow rounded up to 256
 * (HOCCL_ERR_SCRATCH otherwise), and "use_graph" = 1 (HOCCL_ERR_UNSUPPORTED otherwise).
 * Errors: INVALID_ARG (NULL, misaligned, overlapping receive regions, a send region overlapping a receive region),
 * UNSUPPORTED (dtype; handshake mode; a modelled topology without graphs), SCRATCH (modelled topology, staging too small).
 */
hoccl_result_t hoccl_alltoallv(const void* const* send, const size_t* sendcounts, const size_t* sdispls, void* const* recv,
                               const size_t* rdispls, hoccl_dtype_t dtype, hoccl_comm_t comm, hoccl_stream_t stream);

/* ---------------------------------------------------------------- point to point --------------- */

/*
 * Non-blocking matched send/recv between logical ranks (paper Sec. 3.3.2 "Intra-node
 * Communication": a post does not block the caller while the peer has not posted; the transfer
 * happens once both sides are known).  Posts are matched per (src, dst) pair in FIFO order; either
 * side may come first.  The first post parks {buffer, count, dtype, stream} on the host and marks its place in its
 * stream with an event; nothing else is enqueued.  The second post enqueues ONE device-to-device move of count
 * elements that runs after both streams have reached their posts and that both streams then wait for.
 * What this cannot give: work that the FIRST poster enqueues on its stream between its own post and the partner's is
 * not ordered against the transfer (a stream cannot be made to wait, after the fact, for something that is enqueued
 * later): a consumer of the receive buffer, or a writer of the send buffer, must be enqueued after the partner has
 * posted.  Callers that cannot arrange that set "p2p_strict" = 1 (or "handshake" = 1): the post then holds its stream
 * until the transfer is done, whoever posts first, bounded by the watchdog.
 * Mismatch of count or dtype at match time: HOCCL_ERR_MISMATCH from the second call, nothing is
 * enqueued and the parked post is dropped.  Unmatched posts can never hang a stream; their number is
 * hoccl_comm_pending().  Errors: INVALID_ARG (NULL buf, rank out of range, src == dst), CUDA.
 */
hoccl_result_t hoccl_send(const void* buf, size_t count, hoccl_dtype_t dtype, int src, int dst, hoccl_comm_t comm,
                          hoccl_stream_t stream);
hoccl_result_t hoccl_recv(void* buf, size_t count, hoccl_dtype_t dtype, int src, int dst, hoccl_comm_t comm,
                          hoccl_stream_t stream);
int hoccl_comm_pending(hoccl_comm_t comm);
/* First asynchronous failure: handshake mode, as seen by the proxy (OK, TIMEOUT, MISMATCH or CUDA); "fused" and "roles"
 * settings, TIMEOUT if a bounded wait inside the kernel ran out.  clear != 0 resets it. */
hoccl_result_t hoccl_comm_async_error(hoccl_comm_t comm, int clear);
/* Handshake mode: number of stream hand-overs the proxy has served so far. */
long hoccl_comm_handshakes(hoccl_comm_t comm);
/* Handshake mode: how busy the proxy thread is.  *busy_us = time it spent working (launching schedules and moves, writing
 * counters), *span_us = wall time from the first task it accepted to its latest release, since creation or the last reset
 * (reset != 0 zeroes both after reading).  1 - busy / span is the share of the time the thread merely polled: the analogue
 * of the CPU slack the paper reports for its proxy (Sec. 5 "End-to-end workloads").  Both 0 without a proxy. */
hoccl_result_t hoccl_comm_proxy_stats(hoccl_comm_t comm, double* busy_us, double* span_us, int reset);

/* ---------------------------------------------------------------- host-buffer entry points ----- */

/*
 * All-reduce whose buffers are HOST memory (pinned for real asynchrony): h_send[r] / h_recv[r] are
 * host pointers to `count` elements each.  The call copies every h_send[r] into the attached staging
 * memory (needs 2*R*roundup256(count*sizeof(dtype)) bytes), runs the all-reduce there and copies every rank's
 * result back, all ordered on `stream`.  Host-to-device traffic is driven by the copy engines (Sec. 2.3).
 * Pipelined form (default; "host_pieces" > 1 with graphs on): every ring chunk is cut into host_pieces pieces; per
 * piece, the host-to-device copies (2-D copies: that piece of every chunk) run on one internal stream, the ring on that
 * piece (its own cached graph) runs on `stream` as soon as the piece has arrived, and the device-to-host copies follow on
 * a second internal stream, so that the inbound copies, the ring and the outbound copies of different pieces overlap
 * (chunk pipelining, Sec. 3.3.1, applied across the PCIe link); `stream` waits for the last outbound copy.  Chunk boundaries, and therefore every bit of
 * the result, are those of hoccl_allreduce on the whole buffer.  Host buffers of different ranks must not overlap
 * partially (INVALID_ARG); h_recv[r] == h_send[r] is legal.  With host_pieces = 1, use_graph = 0, handshake, onepass,
 * fused or HOCCL_PATH_CE_HOST the three stages run one after the other.
 * Errors: as hoccl_allreduce, SCRATCH if staging is missing or too small.
 */
hoccl_result_t hoccl_host_allreduce(const void* const* h_send, void* const* h_recv, size_t count, hoccl_dtype_t dtype,
                                    hoccl_op_t op, hoccl_comm_t comm, hoccl_stream_t stream);

/* ---------------------------------------------------------------- no-allocation entry point ---- */

/*
 * (The paper has no counterpart: this entry point exists for this library's users only.)
 *
 * hoccl_allreduce_static: the same ring all-reduce as hoccl_allreduce, bit for bit, for callers that
 * are not allowed to allocate device memory and therefore have no scratch to attach to a communicator:
 * for instance a communication thread running beside compute that must never cause the device-wide
 * synchronisation an allocation can imply, or a process whose device memory was handed out once by a
 * static memory planner.  It takes no communicator.  Its ring scratch (inbox and partial slots) is a
 * fixed array of HOCCL_STATIC_SCRATCH_BYTES inside the library image; every GPU that loads the library
 * holds that array until the process exits.  The call itself allocates nothing: no cudaMalloc or
 * cudaFree, no stream, event or graph creation; it only launches kernels on `stream`, in order.
 *
 * send[r] / recv[r]: HOST arrays of R DEVICE pointers to `count` elements each (caller-owned; same
 * in-place and no-overlap rules as hoccl_allreduce).  R: number of logical ranks, 1..64.  `stream` must
 * belong to the device that is current when the call is made.
 *
 * Limits and sharing.  The scratch need is 2 * R * roundup256(ceil(count/R) * sizeof(dtype) + 16) bytes;
 * a call that would need more than HOCCL_STATIC_SCRATCH_BYTES is rejected with HOCCL_ERR_SCRATCH and
 * enqueues nothing (with R = 8 this allows a little under 16 MiB per rank buffer).  All calls on a device
 * share the one array, which keeps whatever the last call left in it; nothing in it has to start at
 * zero, because every byte a sum reads was written by a move of the same call first.  Two calls that
 * overlap in time on the GPU (different streams, no ordering between them) race on the array: order them.
 *
 * First call.  The first call on each device looks up the array's device address (once per device, with
 * that device current) before it launches anything.  If the library's device code has not been loaded on that
 * device yet, this look-up loads it: that is when the device reserves the HOCCL_STATIC_SCRATCH_BYTES of the array,
 * and loading may synchronise the device.  "Allocates nothing" therefore holds from the second call on; make the
 * first call on every device at start-up (a call with a few elements will do), and before any stream capture.
 * The look-up uses the device that is current at the call; `stream` is not checked against it.
 *
 * Errors: INVALID_ARG (NULL or misaligned pointer, overlapping buffers, R out of range), UNSUPPORTED
 * (dtype, op), SCRATCH (beyond the maximum), CUDA (no device, address lookup or launch failed).
 */
#define HOCCL_STATIC_SCRATCH_BYTES (32u << 20)
hoccl_result_t hoccl_allreduce_static(const void* const* send, void* const* recv, size_t count, hoccl_dtype_t dtype,
                                      hoccl_op_t op, int R, hoccl_stream_t stream);

/* ---------------------------------------------------------------- errors and statistics -------- */

const char* hoccl_error_string(hoccl_result_t code);
/* Text of the last CUDA error seen by this communicator ("" if none); valid until the next call. */
const char* hoccl_last_cuda_error(hoccl_comm_t comm);
hoccl_result_t hoccl_last_stats(hoccl_comm_t comm, hoccl_stats_t* out);
hoccl_result_t hoccl_profile_reset(hoccl_comm_t comm);

/* ---------------------------------------------------------------- collective scheduler (host only) --- */

/*
 * The paper's collective scheduler (Sec. 3.4) for a modelled topology: G GPUs in nodes of gpus_per_node (one NVLink
 * domain per node, the RDMA domain between nodes, symmetric peer of GPU u = u ^ 1 inside its node).
 *   C (G x G bytes, row = source)  ->  T = C plus forwarding copies on the (u, u-bar) edges (Eq. 2-4)
 *   ->  stages T^1..T^n by the Birkhoff-like decomposition (Algorithm 1): sum of stages = T (Eq. 5-6), at most one
 *       RDMA flow out of and into every GPU per stage (Eq. 7), stage time tau = max over domains of largest entry /
 *       bandwidth (Eq. 8-9), total = sum of tau (Eq. 10)
 *   ->  per stage and per DMA engine (the source GPU of a copy) a size-weighted interleaving of fixed-size chunks.
 * Pure host code: nothing here touches a device.  bw_* in bytes per second (<= 0 selects 400e9 / 50e9).
 */
typedef struct hoccl_sched* hoccl_sched_t;
typedef enum { HOCCL_FLOW_NATIVE = 0, HOCCL_FLOW_RDMA = 1, HOCCL_FLOW_FWD_SEND = 2, HOCCL_FLOW_FWD_RECV = 3 } hoccl_flow_class_t;
typedef struct {
  int src, dst;                /* the edge this entry uses */
  int cls;                     /* hoccl_flow_class_t */
  int origin_src, origin_dst;  /* the logical flow of C it belongs to */
  uint64_t bytes;
  uint64_t origin_offset;      /* where these bytes start inside the logical flow */
} hoccl_sched_flow_t;

hoccl_result_t hoccl_sched_build(hoccl_sched_t* sched, int G, int gpus_per_node, double bw_nvlink, double bw_rdma,
                                 const uint64_t* C, uint64_t chunk_bytes);
void hoccl_sched_destroy(hoccl_sched_t sched);
int hoccl_sched_num_stages(hoccl_sched_t sched);
double hoccl_sched_stage_tau(hoccl_sched_t sched, int stage);
double hoccl_sched_total_tau(hoccl_sched_t sched);
/* max over RDMA endpoints of their traffic / bw_rdma and over NVLink edges of T / bw_nvlink: no staging can be faster */
double hoccl_sched_lower_bound(hoccl_sched_t sched);
/* which = -2: C, -1: T, s >= 0: the matrix of stage s.  out: G*G entries. */
hoccl_result_t hoccl_sched_matrix(hoccl_sched_t sched, int which, uint64_t* out);
int hoccl_sched_num_flows(hoccl_sched_t sched, int stage);
hoccl_result_t hoccl_sched_get_flow(hoccl_sched_t sched, int stage, int index, hoccl_sched_flow_t* out);
/* the serial chunk queue of one DMA engine in one stage: entry = (flow index in that stage, offset, bytes) */
int hoccl_sched_queue_len(hoccl_sched_t sched, int stage, int gpu);
hoccl_result_t hoccl_sched_queue_get(hoccl_sched_t sched, int stage, int gpu, int index, int* flow, uint64_t* offset,
                                     uint64_t* bytes);

#ifdef __cplusplus
}
#endif
#endif /* HOCCL_H_ */
