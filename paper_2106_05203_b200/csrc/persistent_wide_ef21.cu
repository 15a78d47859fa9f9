// Persistent cluster kernel for EF21 (Algorithm 2), whole-block steps (larger k): instantiations and their lookup.
#define PK_BODY_FILE "persistent_body.inc"
#define PK_KERNEL_NAME persistent_wide_kernel
#define PK_LOOKUP_NAME pk_lookup_wide_ef21
#define PK_PLUS 0
#define PK_EF 0
#define PK_FLOOR 0
#include "persistent_method.inc"
