// Matched send/recv between logical ranks (paper Sec. 3.3.2): host-side FIFO match table, the move is issued when the
// second side posts; in handshake mode the post is handed to the CPU proxy instead.
#include "comm.h"

namespace hoccl {

hoccl_result_t p2p_post(hoccl_comm* c, bool is_send, void* buf, size_t count, int dtype, int src, int dst, cudaStream_t stream) {
  const double t0 = now_us();
  if (!c || !buf) return HOCCL_ERR_INVALID_ARG;
  const size_t e = dtype_size(dtype);
  if (e == 0) return HOCCL_ERR_UNSUPPORTED;
  if (src < 0 || src >= c->R || dst < 0 || dst >= c->R || src == dst) return HOCCL_ERR_INVALID_ARG;
  if ((uintptr_t)buf % e) return HOCCL_ERR_INVALID_ARG;
  if (c->handshake || c->p2p_strict) {
    // the post is handed to the proxy at once; matching happens there, after the stream has reached the post
    if (c->path != HOCCL_PATH_SM) return HOCCL_ERR_UNSUPPORTED;   // see run_collective
    hoccl_result_t rc = ensure_proxy(c);
    if (rc != HOCCL_OK) return rc;
    ProxyTask t;
    t.kind = ProxyTask::P2P;
    t.is_send = is_send;
    t.src = src;
    t.dst = dst;
    t.buf = buf;
    t.count = count;
    t.elem = e;
    t.dtype = dtype;
    t.path = (int)c->path;
    t.copy_ctas = (int)c->copy_ctas;
    CU_TRY(c, cudaSetDevice(c->device));
    CU_TRY(c, c->proxy->submit(stream, t));
    c->stats = hoccl_stats_t{};
    c->stats.n_moves = 1;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  auto key = std::make_pair(src, dst);
  std::deque<Post>& q = c->pending[key];
  if (q.empty() || q.front().is_send == is_send) {
    // No partner yet: the post parks on the host.  Its place in its stream is marked now, so that the move, whenever the
    // partner comes, waits for exactly this point of the stream and not for whatever the stream is given afterwards.
    CU_TRY(c, cudaSetDevice(c->device));
    cudaEvent_t ev = nullptr;
    if (!c->post_events.empty()) {
      ev = c->post_events.back();
      c->post_events.pop_back();
    } else {
      CU_TRY(c, cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
    }
    cudaError_t re = cudaEventRecord(ev, stream);
    if (re != cudaSuccess) {
      c->post_events.push_back(ev);
      return cuda_fail(c, re, "cudaEventRecord (post)");
    }
    q.push_back(Post{is_send, buf, count, dtype, stream, ev});
    c->n_pending++;
    return HOCCL_OK;
  }
  Post peer = q.front();
  q.pop_front();
  c->n_pending--;
  c->post_events.push_back(peer.at_post);   // waits enqueued below capture the record made at post time; the event itself is free again
  if (peer.count != count || peer.dtype != dtype) return HOCCL_ERR_MISMATCH;
  c->stats = hoccl_stats_t{};
  if (count == 0) return HOCCL_OK;
  const void* sbuf = is_send ? buf : peer.buf;
  void* dbuf = is_send ? peer.buf : buf;
  const size_t bytes = count * e;
  if (ranges_overlap((const char*)sbuf, bytes, (const char*)dbuf, bytes)) return HOCCL_ERR_INVALID_ARG;
  CU_TRY(c, cudaSetDevice(c->device));
  const bool two_streams = (peer.stream != stream);
  if (c->path == HOCCL_PATH_CE_HOST) {
    // bounce through pinned host memory: two copy-engine legs, no SM.  All such moves share lane 0 and the start of
    // the staging area, so they run one after the other.
    if (!c->host_staging || bytes > c->host_staging_bytes) return HOCCL_ERR_SCRATCH;
    c->ev_next = 0;
    // ea: where the first poster's stream was when it posted; eb: where this (the second) poster's stream is now
    cudaEvent_t ea = peer.at_post, eb = next_event(c), ed = next_event(c);
    if (!eb || !ed) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    cudaStream_t run = c->lane[0];
    if (two_streams) CU_TRY(c, cudaStreamWaitEvent(run, ea, 0));
    CU_TRY(c, cudaEventRecord(eb, stream));
    CU_TRY(c, cudaStreamWaitEvent(run, eb, 0));
    // Chunk pipelining through the staging area (paper Sec. 3.3.1: one engine fills a staging chunk while the other
    // drains the previous one): the outbound leg of chunk k+1 runs on lane 0 while the inbound leg of chunk k runs on
    // lane 1; PCIe carries both directions at once.
    const size_t chunk = std::max<size_t>((size_t)c->piece_bytes, (size_t)1 << 20);
    if (bytes <= chunk) {
      CU_TRY(c, cudaMemcpyAsync(c->host_staging, sbuf, bytes, cudaMemcpyDeviceToHost, run));
      CU_TRY(c, cudaMemcpyAsync(dbuf, c->host_staging, bytes, cudaMemcpyHostToDevice, run));
    } else {
      cudaStream_t back = c->lane[1];
      cudaEvent_t start = next_event(c);
      if (!start) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(start, run));
      CU_TRY(c, cudaStreamWaitEvent(back, start, 0));   // lane 1 joins after both posting streams, like lane 0
      for (size_t off = 0; off < bytes; off += chunk) {
        const size_t len = std::min(chunk, bytes - off);
        CU_TRY(c, cudaMemcpyAsync(c->host_staging + off, (const char*)sbuf + off, len, cudaMemcpyDeviceToHost, run));
        cudaEvent_t out = next_event(c);
        if (!out) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
        CU_TRY(c, cudaEventRecord(out, run));
        CU_TRY(c, cudaStreamWaitEvent(back, out, 0));
        CU_TRY(c, cudaMemcpyAsync((char*)dbuf + off, c->host_staging + off, len, cudaMemcpyHostToDevice, back));
      }
      cudaEvent_t in_done = next_event(c);
      if (!in_done) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(in_done, back));
      CU_TRY(c, cudaStreamWaitEvent(run, in_done, 0));   // lane 0 stays the serial order of all such moves
    }
    CU_TRY(c, cudaEventRecord(ed, run));
    CU_TRY(c, cudaStreamWaitEvent(peer.stream, ed, 0));
    if (two_streams) CU_TRY(c, cudaStreamWaitEvent(stream, ed, 0));
    c->stats.n_moves = 1;
    c->stats.host_launch_us = now_us() - t0;
    return HOCCL_OK;
  }
  // Large messages on the copy route are cut into up to 4 slices that run on different lanes: one driver copy of
  // 64 MiB reaches ~5.4 TB/s of HBM traffic, two to four concurrent ones ~6.5 TB/s (the same idea as keeping several
  // chunks in flight per connection, paper Sec. 3.3.1 "Multi-QP parallelism").
  int nsplit = 1;
  if (c->path == HOCCL_PATH_CE && bytes >= ((size_t)32 << 20)) {
    nsplit = (int)std::min<size_t>((size_t)c->p2p_split, bytes / ((size_t)16 << 20));
    nsplit = std::max(1, std::min<int>(nsplit, kMaxLanes));
  }
  long n_moves = 0;
  if (!two_streams && nsplit == 1) {
    // both posts came from the same stream: its own order is the whole dependency
    if (c->path == HOCCL_PATH_CE) {
      CU_TRY(c, cudaMemcpyAsync(dbuf, sbuf, bytes, cudaMemcpyDeviceToDevice, stream));
    } else {
      CopyBatch b;
      b.nseg = 1;
      b.pad = 0;
      b.seg[0] = CopySeg{sbuf, dbuf, (unsigned long long)bytes};
      CU_TRY(c, launch_copy(b, (int)c->copy_ctas, stream));
      c->stats.n_move_launches = 1;
      c->stats.max_copy_ctas = c->copy_ctas;
    }
    n_moves = 1;
  } else {
    // the move runs on internal lanes after both posting streams, and both wait for it
    c->ev_next = 0;
    cudaEvent_t ea = peer.at_post, eb = next_event(c);
    if (!eb) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
    CU_TRY(c, cudaEventRecord(eb, stream));
    const size_t slice = ((bytes + nsplit - 1) / nsplit + 255) / 256 * 256;
    for (int i = 0; i < nsplit; i++) {
      const size_t off = (size_t)i * slice;
      if (off >= bytes) break;
      const size_t len = std::min(slice, bytes - off);
      // copy route: rotate lanes so that independent messages overlap; SM copies share one lane so that the CTA
      // budget stays global (two copy kernels never run at the same time)
      cudaStream_t run = c->path == HOCCL_PATH_CE ? c->lane[(c->p2p_rr++) % kMaxLanes] : c->lane[0];
      if (two_streams) CU_TRY(c, cudaStreamWaitEvent(run, ea, 0));
      CU_TRY(c, cudaStreamWaitEvent(run, eb, 0));
      if (c->path == HOCCL_PATH_CE) {
        CU_TRY(c, cudaMemcpyAsync((char*)dbuf + off, (const char*)sbuf + off, len, cudaMemcpyDeviceToDevice, run));
      } else {
        CopyBatch b;
        b.nseg = 1;
        b.pad = 0;
        b.seg[0] = CopySeg{(const char*)sbuf + off, (char*)dbuf + off, (unsigned long long)len};
        CU_TRY(c, launch_copy(b, (int)c->copy_ctas, run));
        c->stats.n_move_launches++;
        c->stats.max_copy_ctas = c->copy_ctas;
      }
      n_moves++;
      cudaEvent_t ed = next_event(c);
      if (!ed) return cuda_fail(c, cudaErrorMemoryAllocation, "event pool");
      CU_TRY(c, cudaEventRecord(ed, run));
      CU_TRY(c, cudaStreamWaitEvent(peer.stream, ed, 0));
      if (two_streams) CU_TRY(c, cudaStreamWaitEvent(stream, ed, 0));
    }
  }
  c->stats.n_moves = n_moves;
  c->stats.host_launch_us = now_us() - t0;
  return HOCCL_OK;
}


}  // namespace hoccl
