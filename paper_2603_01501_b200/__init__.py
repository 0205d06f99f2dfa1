"""B200 (sm_100a) library for the per-step hot path of Gradient Alignment
Control: fused cosine statistics and the in-place rank-one projection with
refresh of the stored direction.  The work is done by the CUDA library behind
``include/gac.h``; this package only binds it (``binding``) and generates
synthetic gradient lists (``synth``)."""
