// Tensor-core projection path (placeholder until the tcgen05 kernel lands: no matrix is
// assigned to it).
#include "kernels.h"

namespace apollo {

bool tensor_path_supports(int, int, int, int) { return false; }
void tensor_path_tiling(int, int, int, int32_t* tiles_n, int32_t* tiles_k) { *tiles_n = 0; *tiles_k = 0; }
int tensor_path_prepare(MatDesc*, int, int, void*, cudaStream_t) { return 0; }
int launch_project_tensor(const MatDesc*, const int*, int, int, const StepParams&, int, int32_t*, cudaStream_t) { return 0; }

}  // namespace apollo
