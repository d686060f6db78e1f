"""B200-native AT-GRPO policy-update hot path: grouped advantages (Eq. 1) and the
clipped-ratio loss through the LM head (Eq. 2), forward and backward, behind the
`libatgrpo.so` C ABI.  `atgrpo` is the thin binding; `workloads` draws synthetic inputs."""
