// Status strings and scratch sizing of the C ABI.
#include <atomic>

#include "twig_common.cuh"

namespace twig {
size_t score_workspace_bytes(int batch, int n_q_heads, int max_len);
size_t tree_attn_stream_workspace_bytes(int batch, int n_q_heads, int max_nodes);
}

static std::atomic<int> g_launch_overlap{1};
bool twig::launch_overlap_enabled() { return g_launch_overlap.load(std::memory_order_relaxed) != 0; }

extern "C" int32_t twig_set_launch_overlap(int32_t on) {
  return g_launch_overlap.exchange(on != 0 ? 1 : 0, std::memory_order_relaxed);
}

extern "C" const char *twig_status_str(twig_status s) {
  switch (s) {
    case TWIG_OK: return "ok";
    case TWIG_ERR_NULL: return "null pointer";
    case TWIG_ERR_SHAPE: return "bad shape";
    case TWIG_ERR_UNSUPPORTED: return "unsupported configuration";
    case TWIG_ERR_WORKSPACE: return "workspace too small";
    case TWIG_ERR_CUDA: return "CUDA error";
    case TWIG_ERR_ALIGN: return "misaligned pointer or stride";
  }
  return "unknown status";
}

extern "C" size_t twig_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim,
                                       int32_t max_len, int32_t max_nodes) {
  (void)head_dim;
  if (batch <= 0 || n_q_heads <= 0 || max_len <= 0) return 0;
  // the larger of the score scratch and the persistent attention kernel's scratch (a buffer serves
  // one of the two, never both)
  const size_t a = twig::score_workspace_bytes(batch, n_q_heads, max_len) + 256;
  const size_t b = twig::tree_attn_stream_workspace_bytes(batch, n_q_heads, max_nodes > 0 ? max_nodes : TWIG_MAX_NODES);
  return a > b ? a : b;
}

extern "C" size_t tree_attention_workspace_bytes(int32_t batch, int32_t n_q_heads, int32_t max_nodes) {
  if (batch <= 0 || n_q_heads <= 0 || max_nodes <= 0) return 0;
  return twig::tree_attn_stream_workspace_bytes(batch, n_q_heads, max_nodes);
}
