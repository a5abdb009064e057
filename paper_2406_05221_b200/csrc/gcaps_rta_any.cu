// gcaps_rta_any.cu -- the kernels that walk all nine size bins in one launch (batches of at most
// 8,192 tasksets) and their launcher, as a translation unit of their own: the device code is the
// one of gcaps_rta.cu, included here with everything else of that file switched off.
#define GCAPS_RTA_ANY_TU 1
#include "gcaps_rta.cu"
