// Instantiations of the Winograd transform kernels (see wino_transforms.cuh).
#include "wino_transforms.cuh"

MNNB_DEFINE_INPUT(12)
MNNB_DEFINE_OUTPUT(12, 6)
