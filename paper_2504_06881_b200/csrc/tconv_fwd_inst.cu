// One (mode, channel combine) family of tiled forward kernels per translation unit, so
// that the families compile in parallel.  Built with -DTCONV_INST_MODE=<tconv_mode_t>
// -DTCONV_INST_CHAN=<1 sum | 2 max | 3 min> -DTCONV_INST_NAME=<exported launcher name>.
#include "tconv_tiled.cuh"
#include "tconv_tiled_bf16.cuh"

#if !defined(TCONV_INST_MODE) || !defined(TCONV_INST_CHAN) || !defined(TCONV_INST_NAME)
#error "TCONV_INST_MODE, TCONV_INST_CHAN and TCONV_INST_NAME must be defined"
#endif

namespace tconv {
int TCONV_INST_NAME(FwdArgs& a) {
    if (a.dtype == TCONV_BF16) return launch_fwd_tiled_bf16_inst<TCONV_INST_MODE, TCONV_INST_CHAN>(a);
    return launch_fwd_tiled_inst<TCONV_INST_MODE, TCONV_INST_CHAN>(a);
}
}  // namespace tconv
