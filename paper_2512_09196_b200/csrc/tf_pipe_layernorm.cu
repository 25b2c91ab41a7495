// Instantiates the V_PIPE kernels of one op (one translation unit per op keeps the build parallel).
#include "tf_pipe.cuh"

namespace tf {
namespace pipe {
PipeFn pipe_fn_layernorm(int dt, int lanes, int vpl, int rpg, bool full) { return pipe_fn_op<OP_LAYERNORM>(dt, lanes, vpl, rpg, full); }
}  // namespace pipe
}  // namespace tf
