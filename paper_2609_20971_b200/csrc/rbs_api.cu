// Host-side pieces shared by the entry points: argument checks, workspace sizes, status strings.
#include "rbs_common.cuh"

namespace rbs {

rbs_status check_shape(const rbs_shape* s) {
  if (s == nullptr) return RBS_ERR_INVALID_ARG;
  if (s->batch <= 0 || s->seqlen <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->block <= 0)
    return RBS_ERR_INVALID_ARG;
  if (s->head_dim != kHeadDim) return RBS_ERR_UNSUPPORTED;
  if (s->block != 64 && s->block != 128 && s->block != 256) return RBS_ERR_UNSUPPORTED;
  if (s->n_q_heads % s->n_kv_heads != 0) return RBS_ERR_UNSUPPORTED;
  if ((s->seqlen + s->block - 1) / s->block > 8192) return RBS_ERR_UNSUPPORTED;
  return RBS_OK;
}

rbs_status check_tensor(const rbs_tensor& t) {
  if (t.ptr == nullptr) return RBS_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(t.ptr) % 16 != 0) return RBS_ERR_INVALID_ARG;
  if (t.stride_batch % 8 != 0 || t.stride_token % 8 != 0 || t.stride_head % 8 != 0) return RBS_ERR_INVALID_ARG;
  if (t.stride_token <= 0 || t.stride_head <= 0 || t.stride_batch < 0) return RBS_ERR_INVALID_ARG;
  return RBS_OK;
}

rbs_status check_chunk(const Dims& x, int q_start_block, int n_q_tokens) {
  if (q_start_block < 0 || n_q_tokens <= 0) return RBS_ERR_INVALID_ARG;
  const long long end = static_cast<long long>(q_start_block) * x.B + n_q_tokens;
  if (end > x.N) return RBS_ERR_INVALID_ARG;
  if (n_q_tokens % x.B != 0 && end != x.N) return RBS_ERR_INVALID_ARG;
  return RBS_OK;
}

SelectWorkspace select_workspace(const Dims& x) {
  SelectWorkspace w;
  w.Mpad = (x.M + 127) / 128 * 128;
  size_t cbytes = static_cast<size_t>(x.L) * x.Hkv * w.Mpad * x.d * sizeof(__nv_bfloat16);
  size_t off = 0;
  w.off_chi = off; off = align_up(off + cbytes, 256);
  w.off_clo = off; off = align_up(off + cbytes, 256);
  w.off_g = off; off = align_up(off + static_cast<size_t>(x.L) * x.Hkv * w.Mpad * sizeof(float), 256);
  w.off_cn = off; off = align_up(off + static_cast<size_t>(x.L) * x.Hkv * w.Mpad * sizeof(float), 256);
  w.off_perm = off; off = align_up(off + static_cast<size_t>(x.L) * x.Hkv * w.Mpad * sizeof(int), 256);
  w.off_counts = off; off = align_up(off + static_cast<size_t>(x.L) * x.Hq * sizeof(unsigned int), 256);
  w.bytes = off;
  return w;
}

// Bounds that hold for every call on a sequence of n_rows query tiles: at most 4 bands, band_rows * bands <= n_rows + 3,
// 24 extra items, 8 split rows and 32 part slots per (band, batch, KV head) group (the constants of rbs_prefill.cu).
PrefillWorkspace prefill_workspace(int L, int Hq, int Hkv, int n_rows, int G) {
  PrefillWorkspace w;
  const size_t groups = static_cast<size_t>(4) * L * Hkv;
  const size_t items = static_cast<size_t>(L) * Hkv * (static_cast<size_t>(n_rows) + 4) * G + groups * 24;
  size_t off = 0;
  w.off_items = off; off = align_up(off + items * 16, 256);
  w.off_splits = off; off = align_up(off + groups * 8 * 16, 256);
  w.off_part_o = off; off = align_up(off + groups * 32 * 128 * 128 * sizeof(float), 256);
  w.off_part_ml = off; off = align_up(off + groups * 32 * 256 * sizeof(float), 256);
  w.bytes = off;
  (void)Hq;
  return w;
}

}  // namespace rbs

extern "C" size_t rbs_workspace_bytes(int op, const rbs_shape* shape) {
  if (rbs::check_shape(shape) != RBS_OK) return 0;
  rbs::Dims x = rbs::make_dims(*shape);
  switch (op) {
    case RBS_OP_SELECT: return rbs::select_workspace(x).bytes;
    case RBS_OP_SELECT_BOX: return rbs::select_box_workspace_bytes(x);
    case RBS_OP_SPARSE_PREFILL:
      return x.B >= 128 ? rbs::prefill_workspace(x.L, x.Hq, x.Hkv, x.M * (x.B / 128), x.G).bytes : 0;
    default: return 0;
  }
}

extern "C" const char* rbs_status_string(rbs_status status) {
  switch (status) {
    case RBS_OK: return "RBS_OK";
    case RBS_ERR_INVALID_ARG: return "RBS_ERR_INVALID_ARG";
    case RBS_ERR_UNSUPPORTED: return "RBS_ERR_UNSUPPORTED";
    case RBS_ERR_WORKSPACE: return "RBS_ERR_WORKSPACE";
    case RBS_ERR_CUDA: return "RBS_ERR_CUDA";
    case RBS_ERR_TIMEOUT: return "RBS_ERR_TIMEOUT";
    case RBS_ERR_DEBUG_CHECK: return "RBS_ERR_DEBUG_CHECK";
  }
  return "RBS_ERR_UNKNOWN";
}

extern "C" const char* rbs_version(void) {
#ifdef RBS_DEBUG
  return "rbs-b200 0.1 (sm_100a, debug checks)";
#else
  return "rbs-b200 0.1 (sm_100a)";
#endif
}
