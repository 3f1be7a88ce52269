// Instantiations of the Winograd transform kernels (see wino_transforms.cuh).
#include "wino_transforms.cuh"

MNNB_DEFINE_INPUT(10)
MNNB_DEFINE_OUTPUT(10, 6)
MNNB_DEFINE_OUTPUT(10, 4)
