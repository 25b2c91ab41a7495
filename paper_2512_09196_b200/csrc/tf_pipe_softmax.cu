// Instantiates the V_PIPE kernels of one op (one translation unit per op keeps the build parallel).
#include "tf_pipe.cuh"

namespace tf {
namespace pipe {
PipeFn pipe_fn_softmax(int dt, int lanes, int vpl, int rpg, bool full) { return pipe_fn_op<OP_SOFTMAX>(dt, lanes, vpl, rpg, full); }
PipeFn pipe_fn_softmax_len(int dt, int lanes, int vpl) { return dt == DT_F32 ? pick_pipe_len<DT_F32>(lanes, vpl) : pick_pipe_len<DT_BF16>(lanes, vpl); }
}  // namespace pipe
}  // namespace tf
