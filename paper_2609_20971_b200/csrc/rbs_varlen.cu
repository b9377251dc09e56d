// rbs_prefill_varlen: a batch of prompts of different lengths packed back to back along the token axis.  Every prompt
// is selected and attended on its own (Sec. 4.1: requests are not concatenated into one causal sequence); this entry
// point runs the three calls of Algorithm 1 per prompt on views of the packed buffers, all in one caller-owned
// workspace that is sized for the longest prompt and reused from prompt to prompt in stream order.
#include "rbs_common.cuh"

namespace rbs {

struct VarlenWorkspace {
  size_t off_centroid, off_radius, off_beta, off_rq, off_mask, off_select, bytes;
};

static VarlenWorkspace varlen_workspace(int max_len, int Hq, int Hkv, int d, int B) {
  rbs_shape sh = {1, max_len, Hq, Hkv, d, B};
  const Dims x = make_dims(sh);
  VarlenWorkspace w;
  size_t off = 0;
  w.off_centroid = off; off = align_up(off + static_cast<size_t>(Hkv) * x.M * d * sizeof(float), 256);
  w.off_radius = off; off = align_up(off + static_cast<size_t>(Hkv) * x.M * sizeof(float), 256);
  w.off_beta = off; off = align_up(off + static_cast<size_t>(Hkv) * x.M * sizeof(float), 256);
  w.off_rq = off; off = align_up(off + static_cast<size_t>(Hkv) * 2 * sizeof(float), 256);
  w.off_mask = off; off = align_up(off + static_cast<size_t>(Hq) * x.M * x.W * sizeof(uint32_t), 256);
  w.off_select = off; off = align_up(off + select_workspace(x).bytes, 256);
  w.bytes = off;
  return w;
}

static rbs_status varlen_check(int n_prompts, const int* cu_seqlens, int Hq, int Hkv, int d, int B, int* max_len) {
  if (n_prompts <= 0 || cu_seqlens == nullptr || cu_seqlens[0] != 0) return RBS_ERR_INVALID_ARG;
  *max_len = 0;
  for (int k = 0; k < n_prompts; ++k) {
    const int len = cu_seqlens[k + 1] - cu_seqlens[k];
    if (len <= 0) return RBS_ERR_INVALID_ARG;
    if (len > *max_len) *max_len = len;
  }
  rbs_shape sh = {1, *max_len, Hq, Hkv, d, B};
  return check_shape(&sh);
}

}  // namespace rbs

extern "C" size_t rbs_varlen_workspace_bytes(int n_prompts, const int* cu_seqlens, int n_q_heads, int n_kv_heads,
                                             int head_dim, int block) {
  int max_len = 0;
  if (rbs::varlen_check(n_prompts, cu_seqlens, n_q_heads, n_kv_heads, head_dim, block, &max_len) != RBS_OK) return 0;
  return rbs::varlen_workspace(max_len, n_q_heads, n_kv_heads, head_dim, block).bytes;
}

extern "C" rbs_status rbs_prefill_varlen(int n_prompts, const int* cu_seqlens, int n_q_heads, int n_kv_heads, int head_dim,
                                         int block, rbs_tensor Q, rbs_tensor K, rbs_tensor V, rbs_tensor O,
                                         float alpha_base, float alpha_rescue, int n_sink, int n_local, int n_recent,
                                         float* density, void* workspace, size_t workspace_bytes, void* stream) {
  using namespace rbs;
  int max_len = 0;
  rbs_status st = varlen_check(n_prompts, cu_seqlens, n_q_heads, n_kv_heads, head_dim, block, &max_len);
  if (st != RBS_OK) return st;
  if ((st = check_tensor(Q)) != RBS_OK || (st = check_tensor(K)) != RBS_OK || (st = check_tensor(V)) != RBS_OK ||
      (st = check_tensor(O)) != RBS_OK)
    return st;
  if (density == nullptr) return RBS_ERR_INVALID_ARG;
  const VarlenWorkspace w = varlen_workspace(max_len, n_q_heads, n_kv_heads, head_dim, block);
  if (workspace == nullptr || workspace_bytes < w.bytes || reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return RBS_ERR_WORKSPACE;
  unsigned char* base = static_cast<unsigned char*>(workspace);
  rbs_stats stats;
  stats.centroid = reinterpret_cast<float*>(base + w.off_centroid);
  stats.radius = reinterpret_cast<float*>(base + w.off_radius);
  stats.beta = reinterpret_cast<float*>(base + w.off_beta);
  stats.rq = reinterpret_cast<float*>(base + w.off_rq);
  uint32_t* mask = reinterpret_cast<uint32_t*>(base + w.off_mask);
  void* sel_ws = base + w.off_select;
  const size_t sel_bytes = w.bytes - w.off_select;
  auto view = [](const rbs_tensor& t, int token0) {   // the prompt's rows of a packed [T][H][d] tensor, as a batch of one
    rbs_tensor v = t;
    v.ptr = static_cast<__nv_bfloat16*>(t.ptr) + static_cast<int64_t>(token0) * t.stride_token;
    v.stride_batch = 0;
    return v;
  };
  for (int k = 0; k < n_prompts; ++k) {
    const int t0 = cu_seqlens[k], len = cu_seqlens[k + 1] - t0;
    rbs_shape sh = {1, len, n_q_heads, n_kv_heads, head_dim, block};
    const rbs_tensor q = view(Q, t0), kk = view(K, t0), v = view(V, t0), o = view(O, t0);
    if ((st = rbs_block_stats(&sh, kk, stats, stream)) != RBS_OK) return st;
    if ((st = rbs_select(&sh, q, stats, alpha_base, alpha_rescue, n_sink, n_local, n_recent, mask,
                         density + static_cast<int64_t>(k) * n_q_heads, nullptr, nullptr, sel_ws, sel_bytes, stream)) != RBS_OK)
      return st;
    if ((st = rbs_sparse_prefill(&sh, q, kk, v, mask, o, nullptr, 0.f, nullptr, 0, stream)) != RBS_OK) return st;
  }
  return RBS_OK;
}
