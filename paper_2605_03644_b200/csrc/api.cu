// Version and error strings of the adapshot C ABI.
#include "common.cuh"

extern "C" const char* adapshot_strerror(int code) {
  switch (code) {
    case ADAPSHOT_OK: return "ok";
    case ADAPSHOT_EINVAL: return "invalid argument (null pointer, non-positive size or unsupported flag)";
    case ADAPSHOT_ESHAPE: return "unsupported shape (head_dim, head ratio, probe list or k out of range)";
    case ADAPSHOT_EALIGN: return "pointer or stride not 16-byte aligned";
    case ADAPSHOT_ECAPACITY: return "capacity too small (ctx_cap, workspace or static scratch)";
    case ADAPSHOT_EUNSUPPORTED: return "dtype or mode not supported by this build";
    case ADAPSHOT_ECUDA: return "a CUDA runtime or driver call failed";
    case ADAPSHOT_EINDEX: return "shot id outside the pool";
    case ADAPSHOT_ETIMEOUT: return "a device pipeline wait exceeded its limit";
    default: return "unknown adapshot error code";
  }
}

extern "C" int adapshot_version(void) { return ADAPSHOT_VERSION_NUMBER; }
