// attend_long.cu (per-group scores + top-U for long sequences) compiled for IEEE-half tensors;
// see attend_f16.cu.
#define SENTRY_ATT_F16 1
#define attend_long_select_supported attend_long_select_f16_supported
#define launch_attend_long_select launch_attend_long_select_f16
#include "attend_long.cu"
