// Status strings and scratch sizing of the C ABI.
#include "twig_common.cuh"

namespace twig {
size_t score_workspace_bytes(int batch, int n_q_heads, int max_len);
}

static bool g_launch_overlap = true;
bool twig::launch_overlap_enabled() { return g_launch_overlap; }

extern "C" int32_t twig_set_launch_overlap(int32_t on) {
  const int prev = g_launch_overlap ? 1 : 0;
  g_launch_overlap = on != 0;
  return prev;
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
  (void)max_nodes;   // tree attention merges its key splits on chip
  if (batch <= 0 || n_q_heads <= 0 || max_len <= 0) return 0;
  return twig::score_workspace_bytes(batch, n_q_heads, max_len) + 256;
}
