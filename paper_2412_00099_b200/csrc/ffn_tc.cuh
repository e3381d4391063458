// Tensor-core (tcgen05 / TMEM / TMA) path of the grouped expert FFN: interface used by api.cu.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace mcce {

// Everything prepared once per weight set: the TMA descriptors of the weight, activation and
// intermediate tensors.  Plain data (the context is zero-initialised as a block of bytes).
struct TcPlan {
  alignas(64) CUtensorMap w_gate, w_up, w_down, sh_gate, sh_up, sh_down;  // weights, 128-row boxes
  alignas(64) CUtensorMap x_routed[2], x_hidden[2], h_all;                // activations, 16-row boxes; two slots
  const void* hidden_ptr[2];   // the hidden tensor x_hidden[slot] was built for
  uint64_t hidden_rows[2];     // and its row count
  int ready;
};

bool tc_applicable(const mcce_config& c);
int tc_plan(const mcce_config& c, const void* Wg, const void* Wu, const void* Wd, const void* shWg, const void* shWu,
            const void* shWd, void* Xg0, void* Xg1, void* H, TcPlan* plan);
// hidden changes from call to call, so its descriptor is (re)built here when the pointer changes.
cudaError_t tc_launch_up(TcPlan& plan, const FfnParams& p, uint32_t* err_flag, cudaStream_t st);
// rows_out: store the expert outputs per (stream, slot) into p.O for a combine pass in slot order (deterministic
// mode) instead of adding w * E_i(x) into p.y with atomics.
cudaError_t tc_launch_down(TcPlan& plan, const FfnParams& p, bool rows_out, uint32_t* err_flag, cudaStream_t st);

}  // namespace mcce
