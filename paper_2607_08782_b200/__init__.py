"""B200-native expert-parallel MoE layer forward under an expert placement
(route -> placement-aware dispatch -> grouped SwiGLU expert FFN -> weighted combine, plus the
placement-cost histograms).  The compute path lives in ``libdirector.so`` (hand-written
sm_100a CUDA behind a C ABI, see ``include/director.h``); ``binding`` marshals arguments only.
"""
