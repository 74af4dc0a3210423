// Instantiations of the send kernel for one (gradient type, state format) pair, chosen with
// -DLOCO_TU_GRAD=<GRAD_*> -DLOCO_TU_STATE=<ST_*>; see loco_dispatch.h.
#include "loco_dispatch.h"

#if !defined(LOCO_TU_GRAD) || !defined(LOCO_TU_STATE)
#error "compile with -DLOCO_TU_GRAD=0|1 -DLOCO_TU_STATE=0|1|2|3"
#endif

namespace loco {

namespace {

template <int GRAD, int STATE, int BITS>
SendKernel pick_send_mode(int mode, int var) {
    if (mode == MODE_FIXED) {
        const int smem = Ring<GRAD, STATE, MODE_FIXED>::kBytes;
        if (var == VAR_LEAN) return {loco_send_kernel<GRAD, STATE, BITS, MODE_FIXED, VAR_LEAN>, smem};
        if (var == VAR_LEAN_NR && (STATE == ST_INT8 || STATE == ST_Q8COMP))
            return {loco_send_kernel<GRAD, (STATE == ST_INT8 || STATE == ST_Q8COMP) ? STATE : ST_INT8, BITS, MODE_FIXED, VAR_LEAN_NR>, smem};
        if (var == VAR_LEAN_X) return {loco_send_kernel<GRAD, STATE, BITS, MODE_FIXED, VAR_LEAN_X>, smem};
        if (var == VAR_LEAN_NR_X && (STATE == ST_INT8 || STATE == ST_Q8COMP))
            return {loco_send_kernel<GRAD, (STATE == ST_INT8 || STATE == ST_Q8COMP) ? STATE : ST_INT8, BITS, MODE_FIXED, VAR_LEAN_NR_X>, smem};
        if (var == VAR_LEAN_SR) return {loco_send_kernel<GRAD, STATE, BITS, MODE_FIXED, VAR_LEAN_SR>, smem};
        if (var == VAR_STOCHASTIC) return {loco_send_kernel<GRAD, STATE, BITS, MODE_FIXED, VAR_STOCHASTIC>, smem};
        return {loco_send_kernel<GRAD, STATE, BITS, MODE_FIXED, VAR_GENERAL>, smem};
    }
    if (STATE == ST_Q8COMP) return {nullptr, 0};                // Q8COMP exists for the global scales only
    constexpr int ST = (STATE == ST_Q8COMP ? ST_FP32 : STATE);
    if (var == VAR_GENERAL) return {loco_send_kernel<GRAD, ST, BITS, MODE_BLOCK, VAR_GENERAL>, Ring<GRAD, ST, MODE_BLOCK>::kBytes};
    if (var == VAR_STOCHASTIC) return {loco_send_kernel<GRAD, ST, BITS, MODE_BLOCK, VAR_STOCHASTIC>, Ring<GRAD, ST, MODE_BLOCK>::kBytes};
    return {loco_send_kernel<GRAD, ST, BITS, MODE_BLOCK, VAR_LEAN>, Ring<GRAD, ST, MODE_BLOCK>::kBytes};
}

}  // namespace

SendKernel LOCO_SEND_TU_NAME(LOCO_TU_GRAD, LOCO_TU_STATE)(int bits, int mode, int var) {
    switch (bits) {
    case 2: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 2>(mode, var);
    case 4: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 4>(mode, var);
    default: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 8>(mode, var);
    }
}

}  // namespace loco
