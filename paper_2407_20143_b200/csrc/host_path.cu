// bcp_reshard_host: the reshard with host buffers.  Pinned buffers are read and written in place
// by the kernels; anything else goes through device staging with uploads, kernels and downloads
// of different target buffers overlapped.
#include "plan_object.hpp"

using namespace bcp;

namespace {

// One-time set-up of the host-buffer path: staging buffers, streams, events, and the work list
// regrouped by target buffer.
int prepare_host_path(bcp_plan_t* p) {
  if (p->s_h2d) return BCP_OK;
  const size_t ns = p->src_bytes.size(), nd = p->dst_bytes.size();
  p->groups.assign(nd, bcp_plan_s::Group());
  std::vector<std::vector<bcp_tile>> tma(nd), big(nd), small(nd), cvt(nd);
  std::vector<std::vector<char>> need(nd, std::vector<char>(ns, 0));
  for (const bcp_tile& t : p->tiles) {
    const uint32_t d = t.dst_buf;
    if (!(t.flags & BCP_TILE_ZERO)) need[d][t.src_buf] = 1;
    bcp_tile u = t;
    u.flags &= ~(BCP_TILE_FOLLOW | (7u << BCP_TILE_FAN_SHIFT));  // groups are per target buffer here: every unit is staged on its own
    ((u.flags & BCP_TILE_CVT_MASK) ? cvt : (u.flags & BCP_TILE_TMA) ? tma : (u.flags & BCP_TILE_SMALL) ? small : big)[d].push_back(u);
  }
  std::vector<bcp_tile> flat;
  flat.reserve(p->tiles.size());
  for (size_t d = 0; d < nd; ++d) {
    bcp_plan_s::Group& g = p->groups[d];
    g.first = flat.size();
    g.n_tma = tma[d].size();
    g.n_big = big[d].size();
    g.n_small = small[d].size();
    g.n_cvt = cvt[d].size();
    flat.insert(flat.end(), tma[d].begin(), tma[d].end());
    flat.insert(flat.end(), big[d].begin(), big[d].end());
    flat.insert(flat.end(), small[d].begin(), small[d].end());
    flat.insert(flat.end(), cvt[d].begin(), cvt[d].end());
    for (uint32_t sb = 0; sb < ns; ++sb)
      if (need[d][sb]) g.needs.push_back(sb);
  }
  // order: always take the target buffer that needs the fewest bytes not yet uploaded, so that
  // the first download starts early and uploads keep running under the downloads
  std::vector<char> have(ns, 0), done(nd, 0);
  for (size_t k = 0; k < nd; ++k) {
    size_t best = nd;
    uint64_t best_cost = ~uint64_t(0);
    for (size_t d = 0; d < nd; ++d) {
      if (done[d]) continue;
      uint64_t cost = 0;
      for (uint32_t sb : p->groups[d].needs)
        if (!have[sb]) cost += p->src_bytes[sb];
      if (cost < best_cost) {
        best_cost = cost;
        best = d;
      }
    }
    done[best] = 1;
    for (uint32_t sb : p->groups[best].needs) have[sb] = 1;
    p->order.push_back(uint32_t(best));
  }
  if (!flat.empty()) {
    BCP_CUDA(cudaMalloc(&p->d_host_tiles, flat.size() * sizeof(bcp_tile)));
    BCP_CUDA(cudaMemcpy(p->d_host_tiles, flat.data(), flat.size() * sizeof(bcp_tile), cudaMemcpyHostToDevice));
  }
  p->stage_src.assign(ns, nullptr);
  p->stage_dst.assign(nd, nullptr);
  for (size_t i = 0; i < ns; ++i) BCP_CUDA(cudaMalloc(&p->stage_src[i], p->src_bytes[i] ? p->src_bytes[i] : 16));
  for (size_t i = 0; i < nd; ++i) BCP_CUDA(cudaMalloc(&p->stage_dst[i], p->dst_bytes[i] ? p->dst_bytes[i] : 16));
  p->ev_src.assign(ns, nullptr);
  p->ev_dst.assign(nd ? nd : 1, nullptr);
  for (cudaEvent_t& e : p->ev_src) BCP_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (cudaEvent_t& e : p->ev_dst) BCP_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  BCP_CUDA(cudaStreamCreateWithFlags(&p->s_d2h, cudaStreamNonBlocking));
  BCP_CUDA(cudaStreamCreateWithFlags(&p->s_h2d, cudaStreamNonBlocking));  // set last: marks the path as ready
  return BCP_OK;
}

}  // namespace

extern "C" {

int bcp_reshard_host(bcp_plan_t* plan, const void* const* src_host, size_t n_src_bufs, void* const* dst_host,
                     size_t n_dst_bufs, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (!plan) return fail(BCP_ERR_INVALID, "plan is NULL");
  if (plan->opt.src_buf_count)  // it writes part of every target buffer; this call hands back whole buffers
    return fail(BCP_ERR_INVALID, "bcp_reshard_host: the plan is restricted to some source buffers (src_buf_count)");
  if (n_src_bufs != plan->src_bytes.size() || n_dst_bufs != plan->dst_bytes.size())
    return fail(BCP_ERR_INVALID, "buffer counts differ from the planned ones");
  if ((n_src_bufs && !src_host) || (n_dst_bufs && !dst_host)) return fail(BCP_ERR_INVALID, "pointer array is NULL");
  for (size_t i = 0; i < n_src_bufs; ++i)
    if (plan->src_bytes[i] && !src_host[i]) return fail(BCP_ERR_INVALID, "source buffer %zu is NULL", i);
  for (size_t i = 0; i < n_dst_bufs; ++i)
    if (plan->dst_bytes[i] && !dst_host[i]) return fail(BCP_ERR_INVALID, "target buffer %zu is NULL", i);
  if (int rc = bind_device(plan)) return rc;
  bcp_plan_t* p = plan;
  // Pinned (or registered) host memory is addressable from the device: then the kernels read the
  // sources and write the targets in place, over PCIe in both directions at once, and no staging
  // copy exists at all.  Anything else goes through device staging buffers.
  {
    std::vector<const void*> dsrc(n_src_bufs, nullptr);
    std::vector<void*> ddst(n_dst_bufs, nullptr);
    bool mapped = true;
    auto device_view = [&](const void* host, void** out) {
      cudaPointerAttributes a;
      if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
        cudaGetLastError();
        return false;
      }
      if (a.type != cudaMemoryTypeHost || !a.devicePointer || (reinterpret_cast<uintptr_t>(a.devicePointer) & 15)) return false;
      *out = a.devicePointer;
      return true;
    };
    for (size_t i = 0; mapped && i < n_src_bufs; ++i)
      if (p->src_bytes[i]) mapped = device_view(src_host[i], const_cast<void**>(&dsrc[i]));
    for (size_t i = 0; mapped && i < n_dst_bufs; ++i)
      if (p->dst_bytes[i]) mapped = device_view(dst_host[i], &ddst[i]);
    if (mapped) {
      // over PCIe every read costs: stage each source piece once and write all its replicas from it
      if (!p->d_fan_tiles && p->n_tma && p->opt.order != 2 && p->opt.fanout != 1) {
        std::vector<bcp_tile> fan(p->tiles.begin(), p->tiles.end());
        mark_followers(fan.data(), p->n_tma);
        BCP_CUDA(cudaMalloc(&p->d_fan_tiles, fan.size() * sizeof(bcp_tile)));
        BCP_CUDA(cudaMemcpy(p->d_fan_tiles, fan.data(), fan.size() * sizeof(bcp_tile), cudaMemcpyHostToDevice));
      }
      for (const Gap& g : p->gaps) memset(static_cast<char*>(dst_host[g.buf]) + g.off, 0, g.len);
      if (int rc = execute(p, dsrc.data(), n_src_bufs, ddst.data(), n_dst_bufs, stream, p->d_fan_tiles)) return rc;
      BCP_CUDA(cudaStreamSynchronize(stream));
      return BCP_OK;
    }
  }
  if (int rc = prepare_host_path(plan)) return rc;
  // device-side pointer table: the staging buffers
  for (size_t i = 0; i < n_src_bufs; ++i) p->h_ptrs[i] = p->stage_src[i];
  for (size_t i = 0; i < n_dst_bufs; ++i) p->h_ptrs[n_src_bufs + i] = p->stage_dst[i];
  if (int rc = upload_tables(p, stream)) return rc;
  p->table_current = false;  // the tables now name the staging buffers, not a caller's
  // The upload stream starts after whatever the caller queued on `stream` before this call.
  BCP_CUDA(cudaEventRecord(p->ev_dst[0], stream));
  BCP_CUDA(cudaStreamWaitEvent(p->s_h2d, p->ev_dst[0], 0));
  std::vector<char> uploaded(n_src_bufs, 0);
  // Target buffers one after the other: upload the sources it still misses, run its units,
  // download it.  Uploads, kernels and downloads sit on three streams, so the download of one
  // target buffer overlaps the uploads for the next (PCIe is full duplex).
  for (uint32_t d : p->order) {
    const bcp_plan_s::Group& g = p->groups[d];
    for (uint32_t sb : g.needs) {
      if (uploaded[sb]) continue;
      uploaded[sb] = 1;
      BCP_CUDA(cudaMemcpyAsync(p->stage_src[sb], src_host[sb], p->src_bytes[sb], cudaMemcpyHostToDevice, p->s_h2d));
      BCP_CUDA(cudaEventRecord(p->ev_src[sb], p->s_h2d));
    }
    if (!p->dst_bytes[d]) continue;
    for (uint32_t sb : g.needs) BCP_CUDA(cudaStreamWaitEvent(stream, p->ev_src[sb], 0));
    BCP_CUDA(cudaMemsetAsync(p->stage_dst[d], 0, p->dst_bytes[d], stream));
    if (int rc = launch_units(p, p->d_host_tiles + g.first, g.n_tma, g.n_big, g.n_small, g.n_cvt, stream)) return rc;
    BCP_CUDA(cudaEventRecord(p->ev_dst[d], stream));
    BCP_CUDA(cudaStreamWaitEvent(p->s_d2h, p->ev_dst[d], 0));
    BCP_CUDA(cudaMemcpyAsync(dst_host[d], p->stage_dst[d], p->dst_bytes[d], cudaMemcpyDeviceToHost, p->s_d2h));
  }
  p->last_stream = stream;
  p->ran = true;
  BCP_CUDA(cudaStreamSynchronize(p->s_h2d));
  BCP_CUDA(cudaStreamSynchronize(stream));
  BCP_CUDA(cudaStreamSynchronize(p->s_d2h));
  return BCP_OK;
}

}  // extern "C"
