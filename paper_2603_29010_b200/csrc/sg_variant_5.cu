// Kernel variant 5 of the contraction kernel (see sg_kernel.cuh: contract_kernel, template parameter kV).
#define SG_VARIANT 5
#include "sg_variant.inc"
