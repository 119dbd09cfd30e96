// Kernel variant 4 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 4
#include "sg_variant.inc"
