// Optional phase timing (tb_profile_enable / tb_profile_read): CUDA events on the launching
// stream around each phase of tb_quantize_layer and of tb_attention_layer.  Process-wide, one
// host thread at a time.
#pragma once

#include "tb_common.cuh"

namespace tb {

enum {
  PH_SETUP = 0, PH_GRID, PH_SWEEP, PH_COMP, PH_CD, PH_OUTPUT, PH_LOSS,   // tb_quantize_layer
  PH_HESSIAN, PH_CROSS, PH_HOUT, PH_FACTOR, PH_PREP, PH_COPY,            // prerequisites (tb_attention_layer)
  PH_COUNT
};
enum { TB_MAX_SPANS = 8192 };
struct PhaseSpan {
  int phase;
  cudaEvent_t a, b;
};
extern bool g_profile_on;
extern PhaseSpan g_spans[TB_MAX_SPANS];
extern int g_n_spans;

struct PhaseScope {
  int idx;
  cudaStream_t st;
  PhaseScope(int phase, cudaStream_t s) : idx(-1), st(s) {
    if (!g_profile_on || g_n_spans >= TB_MAX_SPANS) return;
    PhaseSpan& sp = g_spans[g_n_spans];
    if (cudaEventCreate(&sp.a) != cudaSuccess) return;
    if (cudaEventCreate(&sp.b) != cudaSuccess) {
      cudaEventDestroy(sp.a);
      return;
    }
    sp.phase = phase;
    idx = g_n_spans++;
    cudaEventRecord(sp.a, st);
  }
  ~PhaseScope() {
    if (idx >= 0) cudaEventRecord(g_spans[idx].b, st);
  }
};

}  // namespace tb
