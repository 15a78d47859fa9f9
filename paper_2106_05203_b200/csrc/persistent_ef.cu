// Persistent cluster kernel for the original error feedback method (Algorithm 4), compute warps + service warp.
#define PK_BODY_FILE "persistent_roles.inc"
#define PK_KERNEL_NAME persistent_ef_kernel
#define PK_LOOKUP_NAME pk_lookup_ef
#define PK_PLUS 0
#define PK_EF 1
#define PK_FLOOR 0
#include "persistent_method.inc"
