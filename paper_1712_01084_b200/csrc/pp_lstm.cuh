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

// ---- persistent cell: all steps in one cooperative kernel, gate weights resident in shared memory ----
struct LstmPersistArgs {
    const void* values;          // fragment-ordered tile values of the gate layer (fp16)
    const int32_t* xoff;         // [F] per fragment: element offset of its columns in the pivoted input
    const int32_t* strip_start;  // [S+1]
    const float* bias_piv;       // [M_pad]
    const int32_t* inv_row;      // [M_pad] original gate row -> pivoted row
    const int32_t* inv_col;      // [N_pad] original column of z -> pivoted column
    const void* z;               // [steps + 1][N_pad] fp16: x_t (and h_0 in row 0) in pivoted order, from the prepare kernel
    uint2* g_pk;                 // [2][M_pad] packets {pre-activation bits, step + 1} in pivoted order, buffers
                                 // alternating by step parity; all zero at launch
    int* status;                 // raised to 1 when a bounded wait gave up
    void* h;                     // [H] fp16 out: h_T
    float* c;                    // [H] in: c_0, out: c_T
    int I, H, n_pad, m_pad, steps;
    int n_strips;                // S
    int strips_per_cta;          // power of two <= 16
    unsigned spin_limit;         // re-reads of one packet before a wait gives up (0: the kernel's own limit; set by the launcher)
};

// Shared memory the persistent kernel needs, or 0 when the layer does not qualify (weights of one
// CTA's strips must fit next to two copies of z and one of the pre-activations).  max_frags: most
// fragments any CTA holds.
size_t lstm_persist_smem(int max_frags, int n_pad, int m_pad);
// Cooperative launch of grid CTAs x 512 threads.
cudaError_t launch_lstm_persist(const LstmPersistArgs& a, int grid, size_t smem, cudaStream_t stream);

}  // namespace pp
