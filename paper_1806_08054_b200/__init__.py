"""B200-native ECQ-SGD gradient codec (encode / decode-mean) -- Python binding."""
