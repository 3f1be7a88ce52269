// Instantiations of the Winograd transform kernels (see wino_transforms.cuh).
#include "wino_transforms.cuh"

MNNB_DEFINE_INPUT(3)
MNNB_DEFINE_INPUT(5)
MNNB_DEFINE_INPUT(7)
MNNB_DEFINE_OUTPUT(3, 2)
MNNB_DEFINE_OUTPUT(5, 4)
MNNB_DEFINE_OUTPUT(7, 6)
