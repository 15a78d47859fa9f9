// Persistent cluster kernel for EF21 (Algorithm 2), compute warps + service warp: instantiations and their lookup.
#define PK_BODY_FILE "persistent_roles.inc"
#define PK_KERNEL_NAME persistent_kernel
#define PK_LOOKUP_NAME pk_lookup_ef21
#define PK_PLUS 0
#define PK_EF 0
#define PK_FLOOR 0
#define PK_WITH_SAMPLED 1      // also the instantiations that read sampled rows (Algorithm 5)
#include "persistent_method.inc"
