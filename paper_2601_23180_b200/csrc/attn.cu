#include "host_common.h"
extern "C" size_t trispec_verify_attn_workspace(const trispec_attn_args* a) { (void)a; return 0; }
extern "C" int trispec_verify_attn(const trispec_attn_args* a, void* stream) { (void)a; (void)stream; return TRISPEC_ERR_UNSUPPORTED; }
