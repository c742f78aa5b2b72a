"""B200-native CD-Adam step (communication-compressed distributed AMSGrad, Algorithm 1)."""
