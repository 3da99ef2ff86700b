// The fused forward kernels of hidden width 64 (see dhq_fused.cuh), compiled on their own so that
// the widths build side by side.
#include "dhq_fused.cuh"

namespace dhq {

fused_fn fused_pick_64(bool per_token, bool rot, bool spread, bool ahead) { return pick_width<64, true>(per_token, rot, spread, ahead); }
fused_dump_fn fused_pick_dump_64(bool per_token, bool rot) { return pick_dump_width<64, true>(per_token, rot); }
fused_fn fused_pick_both_64(bool per_token) { return pick_both_width<64>(per_token); }
fused_dump_fn fused_pick_both_dump_64(bool per_token) { return pick_both_dump_width<64>(per_token); }
fused_fn fused_pick_calib_64(bool rot, bool gabor, bool both) { return pick_calib_width<64>(rot, gabor, both); }
fused_fn fused_pick_mixed_64(bool rot, bool ahead) { return pick_mixed_width<64, true>(rot, ahead); }
fused_dump_fn fused_pick_mixed_dump_64(bool rot) { return pick_mixed_dump_width<64, true>(rot); }
fused_fn fused_pick_gabor_64(bool per_token, bool rot) { return pick_gabor_width<64>(per_token, rot); }
fused_dump_fn fused_pick_gabor_dump_64(bool per_token, bool rot) { return pick_gabor_dump_width<64>(per_token, rot); }
fused_fn fused_pick_gabor_both_64(bool per_token) { return pick_gabor_both_width<64>(per_token); }
fused_dump_fn fused_pick_gabor_both_dump_64(bool per_token) { return pick_gabor_both_dump_width<64>(per_token); }

} // namespace dhq
