// The fused forward kernels of hidden width 512 (see dhq_fused.cuh), compiled on their own so that
// the widths build side by side.
#include "dhq_fused.cuh"

namespace dhq {

fused_fn fused_pick_512(bool per_token, bool rot, bool spread, bool ahead) { return pick_width<512, false>(per_token, rot, spread, ahead); }
fused_dump_fn fused_pick_dump_512(bool per_token, bool rot) { return pick_dump_width<512, false>(per_token, rot); }
fused_fn fused_pick_both_512(bool per_token) { return pick_both_width<512>(per_token); }
fused_dump_fn fused_pick_both_dump_512(bool per_token) { return pick_both_dump_width<512>(per_token); }
fused_fn fused_pick_calib_512(bool rot, bool gabor, bool both) { return pick_calib_width<512>(rot, gabor, both); }
fused_fn fused_pick_mixed_512(bool rot, bool ahead) { return pick_mixed_width<512, false>(rot, ahead); }
fused_dump_fn fused_pick_mixed_dump_512(bool rot) { return pick_mixed_dump_width<512, false>(rot); }
fused_fn fused_pick_gabor_512(bool per_token, bool rot) { return pick_gabor_width<512>(per_token, rot); }
fused_dump_fn fused_pick_gabor_dump_512(bool per_token, bool rot) { return pick_gabor_dump_width<512>(per_token, rot); }
fused_fn fused_pick_gabor_both_512(bool per_token) { return pick_gabor_both_width<512>(per_token); }
fused_dump_fn fused_pick_gabor_both_dump_512(bool per_token) { return pick_gabor_both_dump_width<512>(per_token); }

} // namespace dhq
