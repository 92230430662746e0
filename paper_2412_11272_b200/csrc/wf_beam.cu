// Beam-pruning state machine (host-side integer logic; no GPU work).
//
// Sec. 4.2.2: the previous round's transcript is a reference for the current decoding session.
// Decoding starts with beam size 1.  The first comparable top-1 token is searched through the
// reference (search-based alignment); afterwards each comparable top-1 token must equal the next
// reference token to keep the beam at 1; punctuation, timestamp and other special tokens are
// never compared -- neither as the top-1 token nor as reference entries, which the reference
// index passes over; a failed search or a mismatch restores the full beam for the rest of the session.
#include <new>
#include <vector>

#include "../../include/wf_encoder.h"

struct wf_beam_pruner {
  std::vector<int> ref;
  std::vector<unsigned char> special;  // one flag per vocabulary id
  int full_beam;
  long index;       // next reference position to compare with, -1 before alignment
  bool fallen_back;
  long rounds, rounds_at_one;
};

extern "C" {

wf_status wf_beam_pruner_create(const int* reference, int n_reference, const unsigned char* is_special,
                                int vocab_size, int full_beam, wf_beam_pruner** out) {
  if (!out) return WF_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_reference < 0 || (n_reference > 0 && !reference) || vocab_size <= 0 || !is_special || full_beam < 1)
    return WF_ERR_INVALID_ARG;
  for (int i = 0; i < n_reference; ++i)
    if (reference[i] < 0 || reference[i] >= vocab_size) return WF_ERR_INVALID_ARG;
  wf_beam_pruner* p = new (std::nothrow) wf_beam_pruner();
  if (!p) return WF_ERR_INVALID_ARG;
  p->ref.assign(reference, reference + n_reference);
  p->special.assign(is_special, is_special + vocab_size);
  p->full_beam = full_beam;
  p->index = -1;
  p->fallen_back = false;
  p->rounds = p->rounds_at_one = 0;
  *out = p;
  return WF_OK;
}

int wf_beam_pruner_step(wf_beam_pruner* p, int top1_token) {
  if (!p || top1_token < 0 || top1_token >= (int)p->special.size()) return -1;
  int next;
  if (p->fallen_back) {
    next = p->full_beam;
  } else if (p->special[top1_token]) {
    next = 1;
  } else if (p->index < 0) {
    next = p->full_beam;
    p->fallen_back = true;
    for (size_t pos = 0; pos < p->ref.size(); ++pos) {
      if (p->ref[pos] == top1_token) {
        p->index = (long)pos + 1;  // the aligned token counts as matched
        p->fallen_back = false;
        next = 1;
        break;
      }
    }
  } else {
    // the comparison target is the next reference entry that is not itself punctuation, a
    // timestamp or another special token (the previous transcript carries those as well)
    long at = p->index;
    const long n_ref = (long)p->ref.size();
    while (at < n_ref && p->special[p->ref[at]]) ++at;
    if (at < n_ref && p->ref[at] == top1_token) {
      p->index = at + 1;
      next = 1;
    } else {
      p->fallen_back = true;
      next = p->full_beam;
    }
  }
  ++p->rounds;
  if (next == 1) ++p->rounds_at_one;
  return next;
}

wf_status wf_beam_pruner_state(const wf_beam_pruner* p, long* reference_index, int* fallen_back, long* rounds,
                               long* rounds_at_one) {
  if (!p) return WF_ERR_INVALID_ARG;
  if (reference_index) *reference_index = p->index;
  if (fallen_back) *fallen_back = p->fallen_back ? 1 : 0;
  if (rounds) *rounds = p->rounds;
  if (rounds_at_one) *rounds_at_one = p->rounds_at_one;
  return WF_OK;
}

wf_status wf_beam_pruner_destroy(wf_beam_pruner* p) {
  delete p;
  return WF_OK;
}

}  // extern "C"
