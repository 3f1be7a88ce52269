// Instantiations of the Winograd transform kernels (see wino_transforms.cuh).
#include "wino_transforms.cuh"

MNNB_DEFINE_INPUT(8)
MNNB_DEFINE_OUTPUT(8, 6)
MNNB_DEFINE_OUTPUT(8, 4)
MNNB_DEFINE_OUTPUT(8, 2)
