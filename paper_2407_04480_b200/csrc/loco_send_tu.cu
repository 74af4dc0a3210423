// Instantiations of the send kernel for one (gradient type, state format) pair, chosen with
// -DLOCO_TU_GRAD=<GRAD_*> -DLOCO_TU_STATE=<ST_*>; see loco_dispatch.h.
#include "loco_dispatch.h"

#if !defined(LOCO_TU_GRAD) || !defined(LOCO_TU_STATE)
#error "compile with -DLOCO_TU_GRAD=0|1 -DLOCO_TU_STATE=0|1|2|3"
#endif

namespace loco {

namespace {

template <int GRAD, int STATE, int BITS, int MODE, int VAR>
SendKernel both() {
    return {loco_send_kernel<GRAD, STATE, BITS, MODE, VAR>, loco_send_multi_kernel<GRAD, STATE, BITS, MODE, VAR>,
            Ring<GRAD, STATE, MODE>::kBytes};
}

template <int GRAD, int STATE, int BITS>
SendKernel pick_send_mode(int mode, int var) {
    constexpr bool kHasNr = (STATE == ST_INT8 || STATE == ST_Q8COMP);    // only these decompress an 8-bit error
    constexpr int STN = kHasNr ? STATE : ST_INT8;
    constexpr int B2 = BITS == 1 ? 2 : BITS;                              // the sign code has no rounding to randomise
    if (BITS == 1 && var_is_sr(var)) return {nullptr, nullptr, 0};
    if (mode == MODE_FIXED) {
        if (var == VAR_LEAN) return both<GRAD, STATE, BITS, MODE_FIXED, VAR_LEAN>();
        if (var == VAR_LEAN_NR && kHasNr) return both<GRAD, STN, BITS, MODE_FIXED, VAR_LEAN_NR>();
        if (var == VAR_LEAN_X) return both<GRAD, STATE, BITS, MODE_FIXED, VAR_LEAN_X>();
        if (var == VAR_LEAN_NR_X && kHasNr) return both<GRAD, STN, BITS, MODE_FIXED, VAR_LEAN_NR_X>();
        if (var == VAR_LEAN_SR) return both<GRAD, STATE, B2, MODE_FIXED, VAR_LEAN_SR>();
        if (var == VAR_STOCHASTIC) return both<GRAD, STATE, B2, MODE_FIXED, VAR_STOCHASTIC>();
        return both<GRAD, STATE, BITS, MODE_FIXED, VAR_GENERAL>();
    }
    if (STATE == ST_Q8COMP) return {nullptr, nullptr, 0};        // Q8COMP exists for the global scales only
    constexpr int ST = (STATE == ST_Q8COMP ? ST_FP32 : STATE);
    if (var == (VAR_LEAN | VAR_WIDE_BLOCKS)) return both<GRAD, ST, BITS, MODE_BLOCK, VAR_LEAN | VAR_WIDE_BLOCKS>();
    if (var == (VAR_GENERAL | VAR_WIDE_BLOCKS)) return both<GRAD, ST, BITS, MODE_BLOCK, VAR_GENERAL | VAR_WIDE_BLOCKS>();
    if (var == VAR_GENERAL) return both<GRAD, ST, BITS, MODE_BLOCK, VAR_GENERAL>();
    if (var == VAR_STOCHASTIC) return both<GRAD, ST, B2, MODE_BLOCK, VAR_STOCHASTIC>();
    return both<GRAD, ST, BITS, MODE_BLOCK, VAR_LEAN>();
}

}  // namespace

SendKernel LOCO_SEND_TU_NAME(LOCO_TU_GRAD, LOCO_TU_STATE)(int bits, int mode, int var) {
    switch (bits) {
    case 1: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 1>(mode, var);
    case 2: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 2>(mode, var);
    case 4: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 4>(mode, var);
    default: return pick_send_mode<LOCO_TU_GRAD, LOCO_TU_STATE, 8>(mode, var);
    }
}

}  // namespace loco
