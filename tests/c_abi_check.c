/* A plain C11 client of the C ABI: proves that include/tensorcast.h is valid C and that the
 * library can be driven without Python or C++.  It only makes host-side calls (a
 * TC_PLAN_HOST_ONLY plan), so it runs on machines without a GPU.  Prints "ok" on success. */
#include <stdio.h>
#include <string.h>

#include "tensorcast.h"

int main(void)
{
    /* the worked micro-example: L=1, NB=3, B=2, H=2, D=2, E=1, one request of 3 tokens in blocks {2, 0} */
    const int64_t T[1] = {3}, bt_off[2] = {0, 2};
    const int32_t bt[2] = {2, 0};
    tc_plan_spec_t spec;
    memset(&spec, 0, sizeof spec);
    spec.struct_size = (uint32_t)sizeof spec;
    spec.kind = TC_KV_PACK;
    spec.flags = TC_PLAN_HOST_ONLY;
    spec.trace_id = 42;
    spec.kv.L = 1; spec.kv.B = 2; spec.kv.H = 2; spec.kv.D = 2; spec.kv.E = 1;
    spec.kv.src_pool.layout = TC_NHD;
    spec.kv.src_pool.num_blocks = 3;
    spec.kv.src_pool.n_slots = 2;
    spec.kv.packed_layout = TC_HND;
    spec.kv.group.R = 1;
    spec.kv.group.T = T;
    spec.kv.group.bt_off = bt_off;
    spec.kv.group.bt_src = bt;
    tc_plan_t *plan = NULL;
    int rc = tc_plan_create(&spec, &plan);
    if (rc != TC_OK || !plan) { printf("create failed: %s: %s\n", tc_strerror(rc), tc_last_error()); return 1; }
    tc_plan_stats_t st;
    if (tc_plan_stats(plan, &st) != TC_OK || st.trace_id != 42 || st.packed_bytes_required != 24 || st.payload_bytes[0] != 24 || st.executable) {
        printf("unexpected stats\n");
        return 1;
    }
    /* run the lowered descriptors by hand on the example's pool and compare with the hand-derived bytes */
    tc_descriptor_t d[8];
    size_t n = 0;
    if (tc_plan_descriptors(plan, 0, d, 8, &n) != TC_OK || n == 0 || n > 8) { printf("descriptors failed\n"); return 1; }
    unsigned char K[24], V[24], out[24];
    const unsigned char *planes[2] = {K, V};
    for (int i = 0; i < 24; i++) { K[i] = (unsigned char)i; V[i] = (unsigned char)(100 + i); out[i] = 0xCC; }
    for (size_t i = 0; i < n; i++)
        for (uint32_t o = 0; o < d[i].n_outer; o++)
            for (uint32_t k = 0; k < d[i].rows; k++) {
                int64_t a = d[i].src_off + o * d[i].src_outer + (k / d[i].n0) * d[i].src_s1 + (k % d[i].n0) * d[i].src_s0;
                int64_t b = d[i].dst_off + o * d[i].dst_outer + (k / d[i].n0) * d[i].dst_s1 + (k % d[i].n0) * d[i].dst_s0;
                memcpy(out + b, planes[d[i].src_slot + o * d[i].src_slot_step] + a, d[i].run_bytes);
            }
    const unsigned char want_k[12] = {16, 17, 20, 21, 0, 1, 18, 19, 22, 23, 2, 3}; /* NHD pool -> HND packed */
    for (int i = 0; i < 12; i++)
        if (out[i] != want_k[i] || out[12 + i] != want_k[i] + 100) { printf("byte %d differs\n", i); return 1; }
    /* a bad spec is refused with a readable message and no plan */
    spec.kv.E = 3;
    tc_plan_t *bad = (tc_plan_t *)1;
    rc = tc_plan_create(&spec, &bad);
    if (rc != TC_ERR_SHAPE || bad != NULL || strlen(tc_last_error()) == 0) { printf("bad spec not refused\n"); return 1; }
    if (tc_plan_destroy(plan) != TC_OK || tc_plan_destroy(NULL) != TC_OK) return 1;
    printf("ok\n");
    return 0;
}
