#include "csb_device.cuh"
#include "csb_internal.hpp"
namespace csb { void drop_rnn_plans(const csb_matrix*) {} }
extern "C" {
int csb_lstm_forward(int, const csb_matrix_t* const*, const float* const*, const float*, int64_t, int, const float*,
                     const float*, float*, float*, float*, unsigned, void*) { csb::set_error("not built yet"); return CSB_ERR_UNSUPPORTED; }
int csb_gru_forward(int, const csb_matrix_t* const*, const float* const*, const float*, int64_t, int, const float*,
                    float*, float*, unsigned, void*) { csb::set_error("not built yet"); return CSB_ERR_UNSUPPORTED; }
}
