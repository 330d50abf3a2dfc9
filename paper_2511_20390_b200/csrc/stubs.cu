// Tensor-core kernels not written yet: report "unsupported" so that callers fail loudly.
#include "internal.h"
int attention_tc(int, int, int, int, int, const void*, const void*, const void*, void*, uint32_t*, cudaStream_t) { return FREE_ERR_UNSUPPORTED; }
bool attention_tc_supported(int, int) { return false; }
int attention_tc_dpad(int d) { return d; }
