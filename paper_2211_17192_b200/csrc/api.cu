// Error plumbing shared by every entry point of the C ABI.
#include "common.cuh"

namespace spec {

char* error_buffer() {
    static thread_local char buffer[512] = {0};
    return buffer;
}

}  // namespace spec

extern "C" const char* spec_last_error(void) { return spec::error_buffer(); }
