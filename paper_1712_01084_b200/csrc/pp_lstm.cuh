// Launch interface of the LSTM-cell helper kernels (recurrent use of one pivoted gate layer).
#pragma once
#include <cuda_runtime.h>

#include "pp_internal.h"

namespace pp {

struct LstmArgs {
    const int32_t* gather_idx;   // [N_pad] pivoted column -> original column of z = [x_t ; h], -1 = padding
    const int32_t* inv_row;      // [M_pad] original gate row -> pivoted row
    const int32_t* inv_col;      // [N_pad] original column of z -> pivoted column
    void* z;                     // [steps + 1][N_pad] layer inputs in pivoted order, element type of the layer
    const void* x_seq;           // [steps][I]
    void* h;                     // [H] in: h_0, out: h_T (element type of the layer)
    float* c;                    // [H] cell state, updated in place
    const float* g_piv;          // [M_pad] gate pre-activations in pivoted order
    int I, H, n_pad, steps;
    int f16;                     // element type of x_seq / h / z: 1 = binary16, 0 = float
};

// z[t][j] for every step: x_t through the column index array; step 0 also gets h_0; padding is zero.
cudaError_t launch_lstm_prepare(const LstmArgs& a, cudaStream_t stream);
// One cell update from g_piv: c, then h_t into z[t + 1] (pivoted order) and, on the last step, into h.
cudaError_t launch_lstm_gates(const LstmArgs& a, int t, cudaStream_t stream);

}  // namespace pp
