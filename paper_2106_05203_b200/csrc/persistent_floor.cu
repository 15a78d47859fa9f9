// Exchange skeleton of the persistent cluster kernel (no arithmetic of the method), compute warps + service warp.
#define PK_BODY_FILE "persistent_roles.inc"
#define PK_KERNEL_NAME persistent_floor_kernel
#define PK_LOOKUP_NAME pk_lookup_floor
#define PK_PLUS 0
#define PK_EF 0
#define PK_FLOOR 1
#include "persistent_method.inc"
