// placeholder
#include "amla_common.cuh"
namespace amla {
int decode_tc_parts(int sm_count) { return sm_count / 2; }
cudaError_t launch_decode_tc(const DecodeParams&, cudaStream_t, int* unsupported) { *unsupported = 1; return cudaErrorNotSupported; }
}
