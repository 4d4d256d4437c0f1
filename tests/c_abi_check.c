/* A plain C99 program against include/psd.h and libpsd_b200.so: the boundary is usable without C++,
 * without Python and without a GPU for everything that runs on the host (sizes, status texts, argument
 * checks, draft-graph set-up).  Built and run by tests/test_c_header.py. */
#include <stdio.h>
#include <string.h>
#include "psd.h"

int main(void) {
    int failures = 0;
    psd_policy_t p;
    psd_dag_t g;
    uint64_t ranks[3] = {0u, 1u, 3u};      /* root, {sigma_1}, {sigma_1, sigma_2} */
    uint64_t bad[2] = {1u, 0u};            /* node 0 is not the root */
    size_t offsets[15];

    memset(&p, 0, sizeof p);
    p.tau = 0.9f; p.k_min = 1; p.depth = 4;
    failures += strcmp(psd_status_string(PSD_OK), "ok") != 0;
    failures += psd_workspace_bytes(128, 4096, 126464) == 0 || psd_workspace_bytes(128, 4096, 126464) % 256 != 0;
    failures += psd_workspace_bytes(128, 100, 126464) != 0;                    /* H not a multiple of 64 */
    failures += psd_compact_workspace_bytes(128, 4096, 126464) < psd_workspace_bytes(128, 4096, 126464);
    failures += psd_step_host_block(1, 32, 4, offsets) == 0 || offsets[0] != 0 || offsets[14] <= offsets[13];
    failures += psd_dag_init(&g, 3, ranks, NULL) != PSD_OK || g.n_nodes != 3 || g.parents[2] != 3u;
    failures += psd_dag_init(&g, 2, bad, NULL) != PSD_ERR_SHAPE;
    /* argument errors are found on the host, before anything is launched */
    failures += psd_confidence(NULL, NULL, NULL, 128, 4096, 126464, NULL, NULL, NULL, NULL, 0, NULL, NULL) != PSD_ERR_NULL;
    failures += psd_select_unmask(NULL, NULL, NULL, 1, NULL, NULL, 1, 32, p, NULL, NULL, NULL, NULL) != PSD_ERR_NULL;
    failures += strcmp(psd_confidence_kernel_name(128), "confidence_tc_kernel") != 0;
    failures += sizeof(psd_policy_t) != 28;
    printf("%s (%d)\n", failures ? "FAILED" : "ok", failures);
    return failures;
}
