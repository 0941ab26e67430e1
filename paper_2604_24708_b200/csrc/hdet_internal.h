// Helpers shared by the translation units of libhdet (not part of the C ABI).
#pragma once

namespace hdet {

// Stores the text that hdet_last_error(NULL) returns on the calling thread.
void set_handleless_error(const char* msg);

}  // namespace hdet
