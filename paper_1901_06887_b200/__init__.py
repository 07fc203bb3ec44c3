"""Mixed-tenant batched DNN inference on one B200 (sm_100a): C-ABI library + thin binding."""
