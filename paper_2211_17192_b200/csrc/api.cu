// Error plumbing shared by every entry point of the C ABI.
#include <cstdlib>

#include "common.cuh"

namespace spec {

char* error_buffer() {
    static thread_local char buffer[512] = {0};
    return buffer;
}

bool pdl_enabled() {
    static const bool enabled = [] {
        const char* v = std::getenv("SPEC_NO_PDL");
        return !(v && v[0] == '1');
    }();
    return enabled;
}

}  // namespace spec

extern "C" const char* spec_last_error(void) { return spec::error_buffer(); }
