// Development aid, not part of the product interface: per-CTA time stamps of the kernels of a decode step.
//
// Only a library built with -DETA_TIMELINE contains the stamps and exports eta_debug_timeline(); the shipped
// build has neither.  With a device buffer of TL_SLOTS * 8 uint64 registered, every CTA (every warp in the append
// kernel) writes up to eight %globaltimer values (ns) at [k * 8 .. k * 8 + 7], k = region base + CTA index:
//   streaming kernel  TL_DECODE  + c : entry, set-up done, first copy issued, first tile consumed, last tile consumed,
//                                      partials stored, prefix window loaded, dependency wait returned
//   screening kernel  TL_SCREEN  + c ; merge kernel TL_MERGE + c ; predictor TL_PREDICT + c ; append TL_APPEND + row
#pragma once

namespace eta {
constexpr int TL_DECODE = 0;
constexpr int TL_DECODE2 = 256;       // second row of stamps of the streaming kernel (set-up phases)
constexpr int TL_SCREEN = 512, TL_SCREEN_N = 296;
constexpr int TL_MERGE = 808, TL_MERGE_N = 128;
constexpr int TL_PREDICT = 936, TL_PREDICT_N = 32;
constexpr int TL_APPEND = 968, TL_APPEND_N = 48;
constexpr int TL_SLOTS = 1024;
}  // namespace eta

#ifdef ETA_TIMELINE
extern "C" int eta_debug_timeline(void* dev_buffer);   // NULL switches the stamps off (the default)
#endif
