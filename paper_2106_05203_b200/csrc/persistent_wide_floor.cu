// Exchange skeleton of the whole-block persistent kernel (no arithmetic of the method).
#define PK_BODY_FILE "persistent_body.inc"
#define PK_KERNEL_NAME persistent_wide_floor_kernel
#define PK_LOOKUP_NAME pk_lookup_wide_floor
#define PK_PLUS 0
#define PK_EF 0
#define PK_FLOOR 1
#include "persistent_method.inc"
