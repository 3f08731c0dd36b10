// Host-side ends of the path: the keep rate on the target model's tokenisation (Section 3.1) and the assembly
// of the compressed prompt text from character spans (ConcatWithDelim of Algorithm 1, Section 3.2).
// Plain host code; nothing here touches the GPU.
#include <cstring>

#include "common.cuh"

extern "C" double spf_keep_rate(int64_t target_tokens, int64_t budget_tokens) {
  if (target_tokens < 1 || budget_tokens < 1) return 0.0;
  if (budget_tokens >= target_tokens) return 1.0;
  return (double)budget_tokens / (double)target_tokens;
}

extern "C" int64_t spf_snap_budget(int64_t desired_tokens, int64_t block_tokens) {
  if (desired_tokens < 1 || block_tokens < 1) return 0;
  const int64_t blocks = desired_tokens / block_tokens;
  return (blocks < 1 ? 1 : blocks) * block_tokens;
}

extern "C" int64_t spf_concat_with_delim(const char* text, int64_t text_bytes, const int32_t* char_spans, int64_t n_spans,
                                         const char* delim, int64_t delim_bytes, char* out, int64_t out_capacity) {
  using spf::fail;
  spf::clear_error();
  if (text_bytes < 0 || n_spans < 0 || delim_bytes < 0 || out_capacity < 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_concat_with_delim: negative size");
  if ((text == nullptr && text_bytes > 0) || (char_spans == nullptr && n_spans > 0) || (delim == nullptr && delim_bytes > 0) ||
      (out == nullptr && out_capacity > 0))
    return fail(SPF_ERR_INVALID_ARG, "spf_concat_with_delim: null pointer");
  // spans must be ascending and disjoint: then one forward scan of the text finds every byte offset
  int64_t prev_end = 0;
  for (int64_t j = 0; j < n_spans; ++j) {
    const int64_t a = char_spans[2 * j], b = char_spans[2 * j + 1];
    if (a < prev_end || b < a)
      return fail(SPF_ERR_INVALID_ARG, "spf_concat_with_delim: span %lld = [%lld, %lld) is not ascending and disjoint",
                  (long long)j, (long long)a, (long long)b);
    prev_end = b;
  }
  // two passes over the same scan: size first, then (if it fits) the copy
  for (int pass = 0; pass < 2; ++pass) {
    int64_t pos_char = 0, pos_byte = 0, written = 0;
    for (int64_t j = 0; j < n_spans; ++j) {
      const int64_t a = char_spans[2 * j], b = char_spans[2 * j + 1];
      int64_t byte_a = -1, byte_b = -1;
      // advance to character a, then to character b; a character starts at every byte that is not 10xxxxxx
      for (int bound = 0; bound < 2; ++bound) {
        const int64_t want = bound == 0 ? a : b;
        while (pos_char < want && pos_byte < text_bytes) {
          ++pos_byte;
          while (pos_byte < text_bytes && ((unsigned char)text[pos_byte] & 0xC0) == 0x80) ++pos_byte;
          ++pos_char;
        }
        if (pos_char < want)
          return fail(SPF_ERR_INVALID_ARG, "spf_concat_with_delim: span %lld reaches character %lld, the text has %lld",
                      (long long)j, (long long)want, (long long)pos_char);
        (bound == 0 ? byte_a : byte_b) = pos_byte;
      }
      if (j > 0) {
        if (pass == 1) memcpy(out + written, delim, (size_t)delim_bytes);
        written += delim_bytes;
      }
      if (pass == 1) memcpy(out + written, text + byte_a, (size_t)(byte_b - byte_a));
      written += byte_b - byte_a;
    }
    if (pass == 0 && (out == nullptr || written > out_capacity)) return written;
    if (pass == 1) return written;
  }
  return 0;
}
