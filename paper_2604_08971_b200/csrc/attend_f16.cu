// The warp-MMA SentryAttend kernels (fused, streamed, query-block scores) for IEEE-half tensors:
// attend_bf16.cu compiled a second time with fp16 operands in the mixed-precision FMA and the
// warp MMA and fp16 packing (attend_common.cuh), under entry-point names of its own.  In that
// file __nv_bfloat16 is then only the name of a 16-bit storage element.
#define SENTRY_ATT_F16 1
#define attend_bf16_supported attend_f16_supported
#define attend_bf16_gate_fusable attend_f16_gate_fusable
#define launch_attend_bf16 launch_attend_f16
#define attend_long_select_supported attend_long_select_f16_supported
#define launch_attend_long_select launch_attend_long_select_f16
#include "attend_bf16.cu"
