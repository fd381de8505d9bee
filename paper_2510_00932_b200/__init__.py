"""libstreamops for B200: the streaming kernels Copy, Mul (scale), Add, Triad and Dot."""
