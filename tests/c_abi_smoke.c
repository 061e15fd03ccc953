/* A plain C caller of the host-only part of the ABI (no GPU, no CUDA header): the layout
 * arithmetic of Section 3.1 for the short-uniform configuration, whose hand-worked values are in
 * config_sizes.txt (page 262144 B, block 622592 B, 8192 pages, 3449 blocks in a 4 GiB pool). */
#include <stdio.h>

#include "avmp.h"

int main(void)
{
    avmp_model_spec m = {4, 28, 16, 8, 128, 2, 8192 * 16, 8192 * 3, 4};
    avmp_options o;
    avmp_layout l;
    avmp_default_options(&o);
    o.max_requests = 256;
    o.max_pages_per_request = 24;
    if (avmp_derive_layout(&m, 4ull << 30, 0.5, &l) != AVMP_OK) return 1;
    printf("U_kv=%llu U_ssm=%llu kv_cap=%llu ssm_cap=%llu\n", (unsigned long long)l.unit_bytes[0],
           (unsigned long long)l.unit_bytes[1], (unsigned long long)l.cap0[0], (unsigned long long)l.cap0[1]);
    printf("workspace_bytes=%llu\n", (unsigned long long)avmp_workspace_bytes(&m, 4ull << 30, &o));
    printf("%s\n", avmp_error_string(AVMP_ENOSPC));
    /* struct sizes as this compiler sees them: the Python binding must declare the same */
    printf("sizeof avmp_model_spec=%u avmp_options=%u avmp_op=%u avmp_layout=%u avmp_stats=%u avmp_tables=%u "
           "avmp_driver_stats=%u avmp_session_stats=%u\n",
           (unsigned)sizeof(avmp_model_spec), (unsigned)sizeof(avmp_options), (unsigned)sizeof(avmp_op),
           (unsigned)sizeof(avmp_layout), (unsigned)sizeof(avmp_stats), (unsigned)sizeof(avmp_tables),
           (unsigned)sizeof(avmp_driver_stats), (unsigned)sizeof(avmp_session_stats));
    return 0;
}
