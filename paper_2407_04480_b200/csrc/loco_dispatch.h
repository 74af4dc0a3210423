// Kernel selection across translation units.
//
// The kernels are templates (loco_kernels.cuh); instantiating all of them in one translation unit makes the build
// serial and slow, so the instantiations are spread over several object files: loco_send_tu.cu is compiled once per
// (gradient type, state format) and loco_reduce_tu.cu once per (output type, with / without the fused optimizer
// step).  Each object file exports one selection function; the two dispatchers below (loco_api.cu) call the right one.
#pragma once
#include "loco_kernels.cuh"

namespace loco {

using SendFn = void (*)(const SendParams);
using SendMultiFn = void (*)(const SendMultiParams);
struct SendKernel { SendFn fn; SendMultiFn multi_fn; int smem_bytes; };   // one bucket / several buckets per launch; smem_bytes: the cp.async ring

using ReduceFn = void (*)(const ReduceParams);
using ReduceMultiFn = void (*)(const ReduceMultiParams);
struct ReduceKernel { ReduceFn fn; ReduceMultiFn multi_fn; int smem_bytes; };   // multi_fn: several buckets per launch (none with the fused optimizer step); smem_bytes: the cp.async ring (0: none)

#define LOCO_SEND_TU_NAME_(g, s) pick_send_g##g##_s##s
#define LOCO_SEND_TU_NAME(g, s) LOCO_SEND_TU_NAME_(g, s)
#define LOCO_REDUCE_TU_NAME_(o, a) pick_reduce_o##o##_a##a
#define LOCO_REDUCE_TU_NAME(o, a) LOCO_REDUCE_TU_NAME_(o, a)

// one per object file built from loco_send_tu.cu: gradient type g (GRAD_*), state format s (ST_*)
SendKernel pick_send_g0_s0(int bits, int mode, int var);
SendKernel pick_send_g0_s1(int bits, int mode, int var);
SendKernel pick_send_g0_s2(int bits, int mode, int var);
SendKernel pick_send_g0_s3(int bits, int mode, int var);
SendKernel pick_send_g1_s0(int bits, int mode, int var);
SendKernel pick_send_g1_s1(int bits, int mode, int var);
SendKernel pick_send_g1_s2(int bits, int mode, int var);
SendKernel pick_send_g1_s3(int bits, int mode, int var);

// one per object file built from loco_reduce_tu.cu: output type o (GRAD_*), a = 1 with the fused Adam-family step
ReduceKernel pick_reduce_o0_a0(int bits, int mode, int path);
ReduceKernel pick_reduce_o0_a1(int bits, int mode, int path);
ReduceKernel pick_reduce_o1_a0(int bits, int mode, int path);
ReduceKernel pick_reduce_o1_a1(int bits, int mode, int path);

}  // namespace loco
