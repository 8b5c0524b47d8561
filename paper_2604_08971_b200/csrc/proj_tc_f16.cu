// The tcgen05 projection kernels for IEEE-half tensors: proj_tc.cu compiled a second time with
// fp16 operands and packing, under entry-point names of its own.
#define SENTRY_ATT_F16 1
#define project_qkv_tc_supported project_qkv_tc_f16_supported
#define project_out_tc_supported project_out_tc_f16_supported
#define launch_project_qkv_tc launch_project_qkv_tc_f16
#define launch_project_out_tc launch_project_out_tc_f16
#include "proj_tc.cu"
