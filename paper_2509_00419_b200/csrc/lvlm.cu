// Version, status text and workspace sizes of the lvlm library.
#include "common.cuh"

namespace lvlm {
size_t score_tokens_workspace(const lvlm_dims* d);
size_t merge_compact_workspace(const lvlm_dims* d);
size_t kv_compress_workspace(const lvlm_dims* d);
size_t decode_attn_workspace(const lvlm_dims* d);
size_t prefill_attn_workspace(const lvlm_dims* d);
}  // namespace lvlm

// Programmatic dependent launch of the library's kernels is always on in the library proper.  The test build
// (-DLVLM_TEST_HOOKS, a second shared object that only the tests load) can switch it off, to show that
// no result depends on it.
#ifdef LVLM_TEST_HOOKS
static int g_pdl = 1;
extern "C" void lvlm_debug_set_pdl(int on) { g_pdl = on ? 1 : 0; }
namespace lvlm {
bool pdl_enabled() { return g_pdl != 0; }
}  // namespace lvlm
#else
namespace lvlm {
bool pdl_enabled() { return true; }
}  // namespace lvlm
#endif

extern "C" const char* lvlm_version(void) { return "lvlm 0.1 (sm_100a)"; }

extern "C" const char* lvlm_status_string(lvlm_status s) {
    switch (s) {
        case LVLM_OK: return "ok";
        case LVLM_ERR_INVALID_ARG: return "invalid argument";
        case LVLM_ERR_UNSUPPORTED: return "unsupported size or mode";
        case LVLM_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
        case LVLM_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case LVLM_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

extern "C" size_t lvlm_workspace_bytes(int op, const lvlm_dims* d) {
    if (!d) return 0;
    switch (op) {
        case LVLM_OP_SCORE_TOKENS: return lvlm::score_tokens_workspace(d);
        case LVLM_OP_SELECT_TOPK: return 256;          // none needed; a non-zero size keeps callers uniform
        case LVLM_OP_MERGE_COMPACT: return lvlm::merge_compact_workspace(d);
        case LVLM_OP_KV_COMPRESS: return lvlm::kv_compress_workspace(d);
        case LVLM_OP_DECODE_ATTN: return lvlm::decode_attn_workspace(d);
        case LVLM_OP_PREFILL_ATTN: return lvlm::prefill_attn_workspace(d);
    }
    return 0;
}
