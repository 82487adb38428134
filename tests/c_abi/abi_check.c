/* Compiled as plain C against include/ekl_tpo.h and linked with libekl_tpo.so: shows that the
 * header is valid C and that the validation paths answer without any GPU (every call below is
 * rejected, or is a no-op, before anything is enqueued). */
#include <stdio.h>
#include <string.h>

#include "ekl_tpo.h"

static int failures = 0;
#define EXPECT(call, want)                                                             \
    do {                                                                               \
        const ekl_tpo_status got_ = (call);                                            \
        if (got_ != (want)) {                                                          \
            printf("FAIL %s -> %d (%s), wanted %d\n", #call, (int)got_,                \
                   ekl_tpo_status_string(got_), (int)(want));                          \
            ++failures;                                                                \
        }                                                                              \
    } while (0)

int main(void)
{
    static double buf[64];
    static float buf32[64];
    double *p = buf;
    EXPECT(ekl_tpo_inv_helmholtz(p, p, p, p, 0, 4, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_inv_helmholtz(p, p, p, p, 2, -1, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_inv_helmholtz(0, 0, 0, 0, 2, 0, 0), EKL_TPO_OK);
    EXPECT(ekl_tpo_inv_helmholtz(p, 0, p, p, 2, 1, 0), EKL_TPO_ERR_NULL);
    EXPECT(ekl_tpo_inv_helmholtz(p, p, p, p, 100, 1, 0), EKL_TPO_ERR_UNSUPPORTED);
    EXPECT(ekl_tpo_inv_helmholtz(p, p + 16, p + 32, (double *)((char *)p + 4), 2, 1, 0),
           EKL_TPO_ERR_ALIGN);
    EXPECT(ekl_tpo_inv_helmholtz(p, p + 8, p + 16, p + 12, 2, 1, 0), EKL_TPO_ERR_OVERLAP);
    EXPECT(ekl_tpo_inv_helmholtz_f32(buf32, buf32, buf32, buf32, 0, 1, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_inv_helmholtz3(p, p, p, p, p, p, 2, 0, 2, 1, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_inv_helmholtz3(p, p, 0, p, p, p, 2, 2, 2, 1, 0), EKL_TPO_ERR_NULL);
    EXPECT(ekl_tpo_inv_helmholtz3(0, 0, 0, 0, 0, 0, 2, 3, 4, 0, 0), EKL_TPO_OK);
    EXPECT(ekl_tpo_inv_helmholtz_lambda(p, p, p, p, p, 3, 1, 0), EKL_TPO_ERR_UNSUPPORTED);
    EXPECT(ekl_tpo_apply(p, p, p, p, p, 2, 2, 2, 0, 2, 2, 1, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_apply(p, p, p, p, 0, 2, 2, 2, 2, 2, 2, 1, 0), EKL_TPO_ERR_NULL);
    EXPECT(ekl_tpo_apply_f32(buf32, buf32, buf32, buf32, buf32, 1, 1, 1, 1, 1, 1, 0, 0), EKL_TPO_OK);
    EXPECT(ekl_tpo_convection(p, p, p, p, p, 0, 2, 1, 0), EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_inv_helmholtz_host(p, p, p, p, 2, 1, 0, 0, 0), EKL_TPO_ERR_NULL);
    EXPECT(ekl_tpo_inv_helmholtz_host_f32(buf32, buf32, buf32, buf32, 2, -3, buf, 64, 0),
           EKL_TPO_ERR_SHAPE);
    EXPECT(ekl_tpo_apply_host(p, p, p, p, p, 2, 2, 2, 2, 2, 2, 0, 0, 0, 0), EKL_TPO_OK);
    EXPECT(ekl_tpo_inv_helmholtz_host_static(p, p, p, p, 0, 1, 0), EKL_TPO_ERR_SHAPE);
    if (ekl_tpo_host_workspace_bytes(8, 2, 8, 4, 1, 8) == 0) { printf("FAIL workspace size\n"); ++failures; }
    if (ekl_tpo_host_workspace_bytes(0, 2, 8, 4, 1, 8) != 0) { printf("FAIL workspace size 0\n"); ++failures; }
    if (ekl_tpo_version() < 100) { printf("FAIL version\n"); ++failures; }
    if (strcmp(ekl_tpo_status_string(EKL_TPO_OK), "ok") != 0) { printf("FAIL status string\n"); ++failures; }
    printf(failures ? "abi_check: %d failure(s)\n" : "abi_check: ok\n", failures);
    return failures ? 1 : 0;
}
