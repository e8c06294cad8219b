/* A plain-C caller of the library: includes the public header, loads libisv.so at run time and drives a
 * plan-only handle (host bookkeeping, no CUDA call).  Prints the figures the Python test compares. */
#include <dlfcn.h>
#include <stdio.h>
#include <string.h>

#include "isv.h"

#define LOAD(name) \
    name##_t name##_p = (name##_t)dlsym(lib, #name); \
    if (!name##_p) { fprintf(stderr, "missing symbol %s\n", #name); return 2; }

typedef int (*isv_kv_alloc_t)(isv_kv **, const isv_kv_desc *);
typedef int (*isv_kv_free_t)(isv_kv *);
typedef int (*isv_kv_info_t_fn)(isv_kv *, isv_kv_info_t *);
typedef int (*isv_kv_fill_t)(isv_kv *, int32_t, const void *, const void *, const int32_t *, int32_t, int32_t);
typedef int (*isv_kv_append_t)(isv_kv *, int32_t, const void *, const void *, int32_t);
typedef int (*isv_plan_bytes_t)(isv_kv *, int32_t, int32_t, uint64_t *, uint64_t *, uint64_t *, int32_t *);
typedef int (*isv_attn_decode_t)(isv_kv *, int32_t, const void *, void *, float *, const int32_t *, const int32_t *, int32_t);
typedef const char *(*isv_last_error_t)(void);

int main(int argc, char **argv) {
    if (argc < 2) return 2;
    void *lib = dlopen(argv[1], RTLD_NOW | RTLD_LOCAL);
    if (!lib) { fprintf(stderr, "dlopen: %s\n", dlerror()); return 2; }
    LOAD(isv_kv_alloc) LOAD(isv_kv_free) LOAD(isv_kv_fill) LOAD(isv_kv_append) LOAD(isv_plan_bytes)
    LOAD(isv_attn_decode) LOAD(isv_last_error)
    isv_kv_info_t_fn info_p = (isv_kv_info_t_fn)dlsym(lib, "isv_kv_info");
    if (!info_p) return 2;

    isv_kv_desc d;
    memset(&d, 0, sizeof d);
    d.layers = 2; d.q_heads = 8; d.kv_heads = 4; d.head_dim = 128; d.block_tokens = 16; d.dtype = ISV_BF16;
    d.offload_frac = 0.5f; d.max_seqs = 3; d.max_tokens_per_seq = 100; d.plan_only = 1;
    isv_kv *h = NULL;
    if (isv_kv_alloc_p(&h, &d) != ISV_OK || !h) { fprintf(stderr, "alloc: %s\n", isv_last_error_p()); return 1; }
    isv_kv_info_t info;
    if (info_p(h, &info) != ISV_OK) return 1;
    const int32_t lens[3] = {33, 64, 1};
    if (isv_kv_fill_p(h, 0, NULL, NULL, lens, 3, 64) != ISV_OK) return 1;
    if (isv_kv_append_p(h, 0, NULL, NULL, 3) != ISV_OK) return 1;     /* lengths 34, 65, 2 */
    uint64_t res = 0, off = 0, staged = 0;
    int32_t chunks = 0;
    if (isv_plan_bytes_p(h, 0, 3, &res, &off, &staged, &chunks) != ISV_OK) return 1;
    /* compute entry points refuse a plan-only handle with a code and a message, never crash */
    const int rc = isv_attn_decode_p(h, 0, &d, &d, NULL, NULL, NULL, 1);
    printf("block_bytes=%llu kappa=%llu max_blocks=%d res=%llu off=%llu chunks=%d decode_rc=%d err=\"%s\"\n",
           (unsigned long long)info.block_bytes, (unsigned long long)info.kv_bytes_per_token, info.max_blocks_per_seq,
           (unsigned long long)res, (unsigned long long)off, chunks, rc, isv_last_error_p());
    d.head_dim = 96;                                                  /* a bad description is an error code */
    isv_kv *bad = NULL;
    const int rc2 = isv_kv_alloc_p(&bad, &d);
    printf("bad_rc=%d bad_handle=%s\n", rc2, bad ? "set" : "null");
    return isv_kv_free_p(h) == ISV_OK ? 0 : 1;
}
