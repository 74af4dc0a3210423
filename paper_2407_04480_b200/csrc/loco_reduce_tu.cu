// Instantiations of the receive kernels for one output type, with or without the fused Adam-family step, chosen with
// -DLOCO_TU_OUT=<GRAD_*> -DLOCO_TU_ADAM=0|1; see loco_dispatch.h.
#include "loco_dispatch.h"

#if !defined(LOCO_TU_OUT) || !defined(LOCO_TU_ADAM)
#error "compile with -DLOCO_TU_OUT=0|1 -DLOCO_TU_ADAM=0|1"
#endif

namespace loco {

namespace {

template <int OUT, int BITS, int MODE, int PATH>
ReduceKernel both() {
#if LOCO_TU_ADAM
    return {loco_reduce_adam_kernel<OUT, BITS, MODE, PATH>, nullptr, 0};
#else
    return {loco_reduce_kernel<OUT, BITS, MODE, PATH>, loco_reduce_multi_kernel<OUT, BITS, MODE, PATH>,
            static_cast<int>(RecvRing<BITS, MODE>::kCtaBytes)};
#endif
}

template <int OUT, int BITS>
ReduceKernel pick_reduce_path(int mode, int path) {
    if (mode != MODE_FIXED) return both<OUT, BITS, MODE_BLOCK, PATH_MUL>();
    // the sign code has two forms with the global scale: the integer sum (power-of-two s) and d = +-fl(1/s) summed in worker order
    if (BITS == 1) return path == PATH_INT ? both<OUT, BITS, MODE_FIXED, PATH_INT>() : both<OUT, BITS, MODE_FIXED, PATH_MUL>();
    constexpr int B2 = BITS == 1 ? 2 : BITS;        // the division paths are not instantiated for the sign code
    switch (path) {
    case PATH_INT: return both<OUT, B2, MODE_FIXED, PATH_INT>();
    case PATH_MUL: return both<OUT, B2, MODE_FIXED, PATH_MUL>();
    case PATH_NEWTON: return both<OUT, B2, MODE_FIXED, PATH_NEWTON>();
    default: return both<OUT, B2, MODE_FIXED, PATH_DIVIDE>();
    }
}

}  // namespace

ReduceKernel LOCO_REDUCE_TU_NAME(LOCO_TU_OUT, LOCO_TU_ADAM)(int bits, int mode, int path) {
    switch (bits) {
    case 1: return pick_reduce_path<LOCO_TU_OUT, 1>(mode, path);
    case 2: return pick_reduce_path<LOCO_TU_OUT, 2>(mode, path);
    case 4: return pick_reduce_path<LOCO_TU_OUT, 4>(mode, path);
    default: return pick_reduce_path<LOCO_TU_OUT, 8>(mode, path);
    }
}

}  // namespace loco
